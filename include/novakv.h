/*
 * novakv — decode-step attention over a 2-bit, fixed-width, vector-quantised KV cache, and the
 * append-time encoder that fills it (NOVA-KV, arxiv 2608.04074).  C ABI, CUDA sm_100a.
 *
 * Notation (App. A of the paper): row vectors, linear maps act on the right (x R).  B sequences,
 * Hq query heads, Hkv KV heads, Hg = Hq/Hkv, d head dimension, g = 4 coefficients per group,
 * L = d/g groups, C = 256 codewords per group.  Query head h reads KV head h / Hg.
 *
 * Cache format (Sec. 2.2 "Quantization", Sec. 5 "Bit rate"): per token and KV head, L uint8
 * codeword indices for the key and L for the value: 8/g = 2 bits per cached element, no
 * per-token metadata.  Pages hold 64 tokens.  Two caller-owned device pools of equal geometry,
 * uint8 [n_pages][Hkv][64*L] each: one contiguous chunk of 64*L bytes per (page, KV head) for keys
 * and one for values.  Inside a chunk (t = token slot in the page, l = group):
 *     keys    [tile = t/32][plane][t%32][16 bytes]: byte j of a token's L bytes holds the code of group
 *             j ^ (t % 8) for j < 16 and of group j ^ (t % 16) for j >= 16; plane = j / 16.
 *     values  [block = t/16][fr = l%8][fc = t%4][gb = (l/8) ^ (t%2)][b = (t%16)/4].
 * Both orders make every lane of a decode warp load exactly the bytes it consumes with coalesced
 * 128-bit loads, and keep its shared-memory table gathers free of bank conflicts.
 * page_table[seq][i] (int32, row length max_pages_per_seq) names the page of tokens 64i..64i+63.
 *
 * Ownership: the context owns device copies of the calibration tables and one device status
 * word.  Pools, page tables, lengths, queries, outputs and workspaces are the caller's device
 * memory (device pointers unless a parameter says "host").  Calls are asynchronous on `stream`
 * unless stated.  A context is used from one host thread at a time.
 *
 * Errors: every entry point validates its arguments on the host and returns a status; nothing
 * aborts.  Faults only the device can see (page id out of range, length beyond the page table, an
 * appended token that names no valid slot) set bits in the device status word and never trap: a bad
 * page id is replaced by page 0 (every access stays in bounds, the affected sequence's output is
 * unspecified), a bad length is clamped, a bad token is skipped.  Read the word with
 * novakv_last_device_status.  The kernels contain no spin wait.
 *
 * Determinism: for fixed inputs, shapes and device, outputs are bitwise reproducible.
 */
#ifndef NOVAKV_H
#define NOVAKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct novakv_ctx novakv_ctx;        /* opaque */
typedef void* novakv_stream;                 /* a cudaStream_t; NULL is the default stream */

typedef enum {
    NOVAKV_OK = 0,
    NOVAKV_EINVAL = 1,        /* NULL / negative / inconsistent argument */
    NOVAKV_ESHAPE = 2,        /* geometry this build has no kernel for */
    NOVAKV_ENOCALIB = 3,      /* layer has no calibration loaded */
    NOVAKV_EPAGE = 4,         /* page-table geometry inconsistent */
    NOVAKV_EWORKSPACE = 5,    /* workspace NULL or too small */
    NOVAKV_ECUDA = 6,         /* a CUDA runtime call failed */
    NOVAKV_EUNSUPPORTED = 7   /* value codebook off its 7-bit grid, etc. */
} novakv_status;

/* Bits of the device status word. */
#define NOVAKV_DEV_BAD_PAGE      1u   /* a page id was outside [0, n_pages) */
#define NOVAKV_DEV_BAD_LENGTH    2u   /* a sequence length exceeded 64 * max_pages_per_seq */
#define NOVAKV_DEV_WAIT_TIMEOUT  4u   /* reserved: no kernel of this build waits on another thread or copy */
#define NOVAKV_DEV_BAD_TOKEN     8u   /* an appended token named a sequence slot or position out of range */
#define NOVAKV_DEV_SMEM_LAYOUT  16u   /* the scan kernel could not place its tables in shared memory (no output was produced) */

typedef struct {
    int n_layers;
    int n_q_heads;       /* Hq */
    int n_kv_heads;      /* Hkv, divides Hq; Hq/Hkv in {1,2,4,8} */
    int head_dim;        /* d in {64, 128}; (d = 128, Hq/Hkv = 8) is not supported */
    int group_size;      /* must be 4   */
    int codebook_size;   /* must be 256 */
    int page_tokens;     /* must be 64  */
    int device;          /* CUDA device ordinal */
} novakv_config;

/*
 * Calibration tables of one layer (App. B "Bits per element": per (layer, KV head) the three
 * d x d transforms, the mean and L codebooks; value codebooks and a value mean are added here
 * because values are vector-quantised too, App. B "Value quantizer").  HOST pointers, float32,
 * row-major, the equal-volume grouping of Sec. 4 already folded into the columns, so that
 * group l owns coefficient columns [4l, 4l+4).
 *   rk        [Hkv][d][d]   analysis    r = (k - k_mean) rk          (Theorem 1)
 *   rk_inv_t  [Hkv][d][d]   R_K^{-T}    q' = q rk_inv_t; also the synthesis matrix (k^ = r^ rk_inv_t^T + k_mean)
 *   rv        [Hkv][d][d]   orthogonal  s = (v - v_mean) rv,  v^ = s^ rv^T + v_mean   (Corollary 1)
 *   k_mean    [Hkv][d]      may be NULL (= 0)
 *   v_mean    [Hkv][d]      may be NULL (= 0)
 *   cb_k      [Hkv][L][256][4]
 *   cb_v      [Hkv][L][256][4]   every coordinate (head, l, component) on its own 7-bit grid:
 *                                lo + u (hi - lo) / 127, u = 0..127, lo / hi = its smallest / largest value
 *                                over the 256 codewords, evaluated in binary64, rounded once to binary32
 */
typedef struct {
    const float* rk;
    const float* rk_inv_t;
    const float* rv;
    const float* k_mean;
    const float* v_mean;
    const float* cb_k;
    const float* cb_v;
} novakv_calibration;

novakv_status novakv_create(novakv_ctx** out, const novakv_config* cfg);
novakv_status novakv_destroy(novakv_ctx* ctx);
const char* novakv_status_string(novakv_status s);

/*
 * Algorithm 1 lines 1-6 produce these tables offline; this call copies them to the device
 * (synchronous; the caller keeps its memory).  Returns NOVAKV_EUNSUPPORTED if cb_v holds a value
 * off its 7-bit grid (the decode kernel keeps a value codeword as four grid indices; snap the
 * codebooks offline, as the paper does for its own, so that encoder, decoder and any reference agree).
 */
novakv_status novakv_load_calibration(novakv_ctx* ctx, int layer, const novakv_calibration* host);

/* Bytes of one page of the key pool (= of the value pool), all KV heads: Hkv * 64 * L. */
size_t novakv_page_bytes(const novakv_ctx* ctx);

/* Workspace bytes novakv_decode_attention needs for `batch` sequences (device memory, 256-byte aligned). */
size_t novakv_decode_workspace_bytes(const novakv_ctx* ctx, int batch);

/*
 * Write path (Algorithm 1 line 7; Sec. 4 "Complexity"): for each new token t and KV head,
 *     r = (k_t - k_mean) rk,   s = (v_t - v_mean) rv          exact products accumulated in binary64
 * (append-sized batches: blocks of the input dimension in index order, the blocks added pairwise; larger
 * ones: blocks of four input dimensions on the fp64 tensor path; the results differ by less than an ulp of
 * binary64), then for every group l the index of
 * the nearest codeword: exact Euclidean search (Sec. 2.2 "Quantization", App. B "Calibration"), the
 * lowest index winning a tie.  The stored index is the minimiser of the binary64 squared distance
 * sum_i (coef_i - codeword_i)^2 of the binary64 coefficient.  (Both kernels evaluate the 256 distances
 * in binary32 first and keep that result only where the two smallest distances are further apart than
 * binary32 rounding can have moved them; every other group is searched again in binary64.  The result
 * can differ from a binary64 reference only where the two nearest codewords are within ~1e-12 relative.)
 * The 2L index bytes go to page page_table[tok_seq[t]][tok_pos[t]/64] at slot tok_pos[t]%64, and
 * seq_lens[tok_seq[t]] becomes max(seq_lens[tok_seq[t]], tok_pos[t]+1).
 *   k_new, v_new  bf16 [n_tokens][Hkv][d]
 *   tok_seq, tok_pos  int32 [n_tokens]; two tokens of one call must not share (seq, pos);
 *                     tok_seq[t] = -1 marks an unused entry of the list: it is skipped, no status bit
 *   n_tokens = 0 is a no-op.  Out-of-range tokens/pages set device status bits and are skipped.
 */
novakv_status novakv_encode_append(novakv_ctx* ctx, int layer,
    const void* k_new, const void* v_new, const int32_t* tok_seq, const int32_t* tok_pos,
    int n_tokens, uint8_t* k_pages, uint8_t* v_pages, int n_pages,
    const int32_t* page_table, int max_pages_per_seq, int n_seq, int32_t* seq_lens,
    novakv_stream stream);

/*
 * Read path (Algorithm 1 line 8; App. B "Decoding kernel and read path"): one decode step for
 * `batch` sequences directly on the index cache, never materialising keys or values:
 *     q'_h = q_h rk_inv_t                                     one d x d product per head
 *     z_hj = sm_scale * sum_l < q'_h[4l..4l+3], cb_k[l][kidx_j[l]] >     (k_mean dropped: Lemma S1)
 *     p_h  = softmax_j(z_hj)  over positions 0 .. seq_lens[b]-1
 *     o_h  = ( sum_j p_hj concat_l cb_v[l][vidx_j[l]] ) rv^T + v_mean    (Remark after Corollary 1)
 * computed split over the sequence with an exact log-sum-exp merge, binary32 accumulation.
 *   q    bf16 [batch][Hq][d]
 *   out  [batch][Hq][d], float32 if out_is_fp32 else bf16; a sequence of length 0 yields zeros
 *   workspace  at least novakv_decode_workspace_bytes(ctx, batch) bytes; contents are scratch
 */
novakv_status novakv_decode_attention(novakv_ctx* ctx, int layer, const void* q,
    const uint8_t* k_pages, const uint8_t* v_pages, int n_pages,
    const int32_t* page_table, int max_pages_per_seq, const int32_t* seq_lens, int batch,
    float sm_scale, void* out, int out_is_fp32, void* workspace, size_t workspace_bytes,
    novakv_stream stream);

/*
 * Key format with a per-token scale (Algorithm 3, the "Normalize" step; App. B "Decoding kernel and
 * read path": the read kernel fetches rho_j from per-token metadata and applies it with a single multiply;
 * Sec. 5 "Bit rate": one BF16 scale per token and KV head, 16/d extra bits per key element, 2.125 at
 * d = 128).  The key codebooks of the layer must have been trained on normalised coefficients.
 *   write:  r as in novakv_encode_append (binary32 coefficients);
 *           rho = bf16( float( sqrt( sum_i r_i^2 / d ) ) ), the sum and the root in binary64, both
 *           roundings to nearest even (the order of the binary64 sum is not specified); a rho that is
 *           not positive and finite is replaced by 1;  n_i = r_i / rho in binary32 (IEEE division);
 *           the codeword search runs on n as in novakv_encode_append.  Values are not scaled.
 *   read:   z_hj = rho_j * sm_scale * sum_l < q'_h[4l..4l+3], cb_k[l][kidx_j[l]] >, the rest as in
 *           novakv_decode_attention.
 *   k_scales  device, bf16 [n_pages][Hkv][64]: the scale of the token in slot s of page p, KV head h,
 *             at (p * Hkv + h) * 64 + s; novakv_scale_page_bytes() = Hkv * 64 * 2 bytes per page.
 * Other arguments, ownership and errors are those of the unscaled calls; NOVAKV_EUNSUPPORTED if the
 * CUDA-core value path was selected with novakv_debug_set_value_path.
 */
size_t novakv_scale_page_bytes(const novakv_ctx* ctx);
novakv_status novakv_encode_append_scaled(novakv_ctx* ctx, int layer,
    const void* k_new, const void* v_new, const int32_t* tok_seq, const int32_t* tok_pos,
    int n_tokens, uint8_t* k_pages, uint8_t* v_pages, void* k_scales, int n_pages,
    const int32_t* page_table, int max_pages_per_seq, int n_seq, int32_t* seq_lens,
    novakv_stream stream);
novakv_status novakv_decode_attention_scaled(novakv_ctx* ctx, int layer, const void* q,
    const uint8_t* k_pages, const uint8_t* v_pages, const void* k_scales, int n_pages,
    const int32_t* page_table, int max_pages_per_seq, const int32_t* seq_lens, int batch,
    float sm_scale, void* out, int out_is_fp32, void* workspace, size_t workspace_bytes,
    novakv_stream stream);

/*
 * Decode step with a learned attention sink (App. "Attention sinks in the quantized serving path"):
 * an extra logit sink_logits[h] per query head that enters the softmax normaliser and has no value,
 *     p_hj = exp(z_hj) / ( sum_i exp(z_hi) + exp(sink_h) ),   o_h = sum_j p_hj v^_j.
 * The sink term is added exactly once, after the cross-split merge.  Because the read path drops the
 * constant q_h . k_mean * sm_scale from every token logit (Lemma S1 no longer applies with a sink),
 * the kernel shifts the sink logit by the same constant (one d-dimensional dot product per head and
 * step), and v_mean enters with the token mass sum_j p_hj instead of 1.
 *   sink_logits  device, float32 [Hq], natural-log units (the units of q.k * sm_scale)
 *   k_scales     NULL for the 2-bit key format, else the scale pool of novakv_encode_append_scaled
 * Other arguments, results and errors are those of novakv_decode_attention; a sequence of length 0
 * yields zeros.
 */
novakv_status novakv_decode_attention_sink(novakv_ctx* ctx, int layer, const void* q,
    const uint8_t* k_pages, const uint8_t* v_pages, const void* k_scales, const float* sink_logits,
    int n_pages, const int32_t* page_table, int max_pages_per_seq, const int32_t* seq_lens, int batch,
    float sm_scale, void* out, int out_is_fp32, void* workspace, size_t workspace_bytes,
    novakv_stream stream);

/*
 * Decode step on a cache with a BF16 sink-plus-recent band (Sec. 5 "Baselines"; App. B "Sink-plus-recent
 * band" and its figure "Cache layout at decoding position t"): the first n_sink tokens and the most
 * recent tokens of a sequence are held exactly in bf16 and excluded from quantisation; the tokens in
 * between are read from the index cache.  The softmax runs over all of them: the band contributes one
 * more partial (max, sum, sum_j p_j v_j in the original value domain) to the exact merge.
 *   index cache  positions n_sink .. n_sink + quant_lens[b] - 1 of sequence b (page column n_sink/64
 *                onwards of its page-table row); quant_lens device int32 [batch]; n_sink a multiple of 64
 *   band_k, band_v  device bf16 [batch][band_cap][Hkv][d].  Of sequence b, slots 0 .. sink_cnt-1 hold
 *                its first tokens, and slots n_sink + (ring_start + i) % (band_cap - n_sink),
 *                i < ring_len, its most recent ones (a ring: App. B has a new token join the recent band
 *                first and leaves quantisation to batches of eight decode steps - the caller appends to
 *                the ring and, when it has grown by eight, passes the eight oldest to
 *                novakv_encode_append[_scaled] and advances ring_start and quant_lens)
 *   band_meta    device int32 [batch][3] = (sink_cnt, ring_start, ring_len); values are clamped to the
 *                buffer
 *   k_scales, sink_logits  NULL or as in novakv_decode_attention_scaled / _sink
 * A sequence with no token at all yields zeros.  Other arguments and errors as novakv_decode_attention.
 */
novakv_status novakv_decode_attention_banded(novakv_ctx* ctx, int layer, const void* q,
    const uint8_t* k_pages, const uint8_t* v_pages, const void* k_scales, const float* sink_logits,
    int n_pages, const int32_t* page_table, int max_pages_per_seq, const int32_t* quant_lens,
    const void* band_k, const void* band_v, int band_cap, int n_sink, const int32_t* band_meta,
    int batch, float sm_scale, void* out, int out_is_fp32, void* workspace, size_t workspace_bytes,
    novakv_stream stream);

/*
 * Write side of the BF16 band (App. B "Sink-plus-recent band": a new token joins the recent band first;
 * quantisation is deferred and happens for `block` tokens at a time, eight in the paper): one new token
 * for every sequence, all bookkeeping in device memory, no host synchronisation.  For sequence b with
 * band_meta[b] = (sink_cnt, ring_start, ring_len) and ring_cap = band_cap - n_sink:
 *   - sink_cnt < n_sink: the token goes to slot sink_cnt, sink_cnt grows by one;
 *   - otherwise it goes to ring slot n_sink + (ring_start + ring_len) % ring_cap and ring_len grows by one;
 *     if ring_len has reached n_rec + block, the `block` oldest ring tokens are encoded into the index cache
 *     at positions n_sink + quant_lens[b] .. + block - 1 (the encoder of the format the optional pools
 *     select: k_scales != NULL the scaled key format, v_meta != NULL as well the deployed format), then
 *     ring_start = (ring_start + block) % ring_cap, ring_len -= block, quant_lens[b] += block, and
 *     seq_lens[b] (the index cache's own length, as novakv_encode_append maintains it) follows.
 * The tokens leaving the band are staged in `staging` together with their (sequence, position) list;
 * sequences that flush nothing contribute unused entries.
 *   k_new, v_new   device bf16 [batch][Hkv][d]
 *   band_k, band_v, band_meta, quant_lens   as in novakv_decode_attention_banded, read and written
 *   n_rec, block   > 0 with n_rec + block <= band_cap - n_sink; n_sink a multiple of 64
 *   staging        device, novakv_band_append_staging_bytes(ctx, batch, block) bytes, 256-byte aligned
 * Returns NOVAKV_EINVAL for inconsistent sizes, NOVAKV_EWORKSPACE for a short or misaligned staging buffer.
 */
size_t novakv_band_append_staging_bytes(const novakv_ctx* ctx, int batch, int block);
novakv_status novakv_band_append(novakv_ctx* ctx, int layer, const void* k_new, const void* v_new, int batch,
    void* band_k, void* band_v, int band_cap, int n_sink, int n_rec, int block,
    int32_t* band_meta, int32_t* quant_lens,
    uint8_t* k_pages, uint8_t* v_pages, void* k_scales, void* v_meta, int n_pages,
    const int32_t* page_table, int max_pages_per_seq, int32_t* seq_lens,
    void* staging, size_t staging_bytes, novakv_stream stream);

/*
 * The paper's deployed cache format (Sec. 5 "Bit rate": keys at 2.125 bits per element; values as 2-bit
 * integers with one BF16 scale and one BF16 zero-point per token, 2 + 32/128 = 2.25 bits per element;
 * App. B read path: the 2-bit codes are dequantised in a rotation basis): keys as in
 * novakv_encode_append_scaled; values scalar
 * quantised to 2 bits in the Corollary 1 basis R_V (which stands in for the rotation the paper takes from
 * prior work), one bf16 (scale, zero) pair per token and KV head:
 *     s = (v - v_mean) rv                      binary32 coefficients, as in novakv_encode_append
 *     zero  = bf16(min_i s_i)
 *     scale = bf16((max_i s_i - zero) / 3)     in binary32; replaced by 1 if not positive and finite
 *     code_i = clamp(rint((s_i - zero) / scale), 0, 3)      binary32 subtraction and division, ties to even
 *     read:  s^_i = zero + scale * code_i,  o_h = (sum_j p_hj s^_j) rv^T + v_mean
 * The byte of group l in the value pool holds code_{4l} | code_{4l+1} << 2 | code_{4l+2} << 4 |
 * code_{4l+3} << 6, at the position the vector-quantised format gives that group's index; cb_v of the
 * calibration is not used.
 *   v_meta  device, bf16 [n_pages][Hkv][64][2] = (scale, zero); novakv_value_meta_page_bytes() per page
 * novakv_decode_attention_deployed takes the arguments of novakv_decode_attention_banded plus v_meta;
 * band_k = band_v = band_meta = NULL reads the whole sequence from the index cache (quant_lens are then
 * the sequence lengths, n_sink and band_cap are ignored); sink_logits may be NULL.
 */
size_t novakv_value_meta_page_bytes(const novakv_ctx* ctx);
novakv_status novakv_encode_append_deployed(novakv_ctx* ctx, int layer,
    const void* k_new, const void* v_new, const int32_t* tok_seq, const int32_t* tok_pos,
    int n_tokens, uint8_t* k_pages, uint8_t* v_pages, void* k_scales, void* v_meta, int n_pages,
    const int32_t* page_table, int max_pages_per_seq, int n_seq, int32_t* seq_lens,
    novakv_stream stream);
novakv_status novakv_decode_attention_deployed(novakv_ctx* ctx, int layer, const void* q,
    const uint8_t* k_pages, const uint8_t* v_pages, const void* k_scales, const void* v_meta,
    const float* sink_logits, int n_pages, const int32_t* page_table, int max_pages_per_seq,
    const int32_t* quant_lens, const void* band_k, const void* band_v, int band_cap, int n_sink,
    const int32_t* band_meta, int batch, float sm_scale, void* out, int out_is_fp32, void* workspace,
    size_t workspace_bytes, novakv_stream stream);

/*
 * The same decode step for callers that cannot supply a workspace and cannot allocate one: an
 * engine that gave all device memory to its own pool, a plug-in inside it, a serving loop that must
 * never call cudaMalloc (the call synchronises the device).  (The paper has no counterpart; this is
 * a property of the library, not of the method.)  The scratch that novakv_decode_attention takes as
 * `workspace` is a fixed array of NOVAKV_NOALLOC_SCRATCH_BYTES inside the library's device image:
 * every GPU that loads the library holds it until the process exits.
 *   - Arguments and results are those of novakv_decode_attention without workspace/workspace_bytes.
 *   - Returns NOVAKV_EWORKSPACE when novakv_decode_workspace_bytes(ctx, batch) exceeds
 *     NOVAKV_NOALLOC_SCRATCH_BYTES; the workspace grows with the batch and with the number of SMs of the
 *     device (for the Qwen3-8B shape on a 148-SM device the largest batch that fits is 77 sequences).
 *   - Calls no cudaMalloc, cudaFree or other allocating routine, and records no timing events.
 *   - All calls on a device share the array: calls that overlap on the GPU (other streams, other
 *     contexts) race; calls on one stream are ordered and safe.  Every scratch word is written
 *     before it is read within a call, so nothing needs clearing between calls.
 *   - The first call on each device queries the array's device address (a synchronous runtime
 *     call); issue that first call before any stream capture begins.  The address is cached per device
 *     in a process-wide table that is written without a lock: the look-up gives the same value every
 *     time, so concurrent first calls are harmless, but a context is still used from one thread at a time.
 */
#define NOVAKV_NOALLOC_SCRATCH_BYTES (4u << 20)
novakv_status novakv_decode_attention_noalloc(novakv_ctx* ctx, int layer, const void* q,
    const uint8_t* k_pages, const uint8_t* v_pages, int n_pages,
    const int32_t* page_table, int max_pages_per_seq, const int32_t* seq_lens, int batch,
    float sm_scale, void* out, int out_is_fp32, novakv_stream stream);

/* Synchronises `stream`, returns the device status word in *word and clears it. */
novakv_status novakv_last_device_status(novakv_ctx* ctx, novakv_stream stream, uint32_t* word);

/*
 * One serving step from HOST buffers (Fig. 1(b): write path then read path): copies the new
 * tokens and the queries to the device, appends, decodes and copies the output back, all on
 * `stream`, then synchronises it.  The index cache itself stays resident on the device.
 *   k_new_host, v_new_host  bf16 [n_tokens][Hkv][d];  tok_seq_host, tok_pos_host int32 [n_tokens]
 *   q_host   bf16 [batch][Hq][d];  out_host  float32 [batch][Hq][d]
 *   staging  device scratch of novakv_step_staging_bytes(ctx, batch, n_tokens) bytes
 * A buffer in page-locked (pinned, device-mapped) host memory is read or written by the kernels
 * directly across the bus; any other host buffer is staged through `staging` with a copy on `stream`.
 * Either way the step's inputs travel host -> device and its output device -> host inside the call.
 * novakv_step_host_async enqueues the same work and returns without waiting: the host buffers must stay
 * valid and out_host must not be read until `stream` has been synchronised (or an event recorded behind
 * the call has completed); novakv_step_host is that call followed by the synchronisation.
 */
size_t novakv_step_staging_bytes(const novakv_ctx* ctx, int batch, int n_tokens);
novakv_status novakv_step_host_async(novakv_ctx* ctx, int layer,
    const void* k_new_host, const void* v_new_host, const int32_t* tok_seq_host,
    const int32_t* tok_pos_host, int n_tokens, const void* q_host,
    uint8_t* k_pages, uint8_t* v_pages, int n_pages, const int32_t* page_table,
    int max_pages_per_seq, int32_t* seq_lens, int batch, float sm_scale, float* out_host,
    void* staging, size_t staging_bytes, void* workspace, size_t workspace_bytes,
    novakv_stream stream);
novakv_status novakv_step_host(novakv_ctx* ctx, int layer,
    const void* k_new_host, const void* v_new_host, const int32_t* tok_seq_host,
    const int32_t* tok_pos_host, int n_tokens, const void* q_host,
    uint8_t* k_pages, uint8_t* v_pages, int n_pages, const int32_t* page_table,
    int max_pages_per_seq, int32_t* seq_lens, int batch, float sm_scale, float* out_host,
    void* staging, size_t staging_bytes, void* workspace, size_t workspace_bytes,
    novakv_stream stream);

/* ---- measurement and staged-parity helpers (not part of the serving contract) ---------------- */

/*
 * Search only (second half of the write path): coefficients are given, float32 [n][Hkv][d]
 * (device); writes logical indices uint8 [n][Hkv][L] (device).  which = 0 keys, 1 values.
 */
novakv_status novakv_search_coefficients(novakv_ctx* ctx, int layer, int which, const float* coef,
    int n, uint8_t* idx_out, novakv_stream stream);

/*
 * Uncompressed comparator: the same decode step on a bf16 paged cache
 * (pools bf16 [n_pages][Hkv][64][d] for keys and for values), textbook attention with the same
 * split-and-merge structure.  Used to report the compression speed-up on identical shapes.
 * window > 0 restricts attention to the last `window` positions (sliding-window layers).
 */
size_t novakv_bf16_workspace_bytes(const novakv_ctx* ctx, int batch, int max_pages_per_seq);
novakv_status novakv_bf16_decode_attention(novakv_ctx* ctx, const void* q,
    const void* k_pages_bf16, const void* v_pages_bf16, int n_pages,
    const int32_t* page_table, int max_pages_per_seq, const int32_t* seq_lens, int batch,
    float sm_scale, int window, void* out, int out_is_fp32, void* workspace,
    size_t workspace_bytes, novakv_stream stream);

/*
 * Per-kernel device timing for roofline accounting: when enabled, the library brackets the
 * dominant kernel of each decode / append call with CUDA events on the call's stream.
 * novakv_profile_read synchronises, returns the accumulated milliseconds and launch counts since
 * the last read and resets them.  kind: 0 = decode stage 1 (index scan), 1 = encode kernel,
 * 2 = bf16 comparator stage 1.
 */
novakv_status novakv_profile_enable(novakv_ctx* ctx, int on);
novakv_status novakv_profile_read(novakv_ctx* ctx, int kind, double* total_ms, long* launches);

/*
 * Test knob: number of CTAs the decode scan kernel is launched with (0 = one per SM, the default;
 * values above the SM count are clamped).  The result must not depend on it beyond binary32
 * rounding, because the split over the sequence is merged exactly (App. B, two-stage split-KV).
 */
novakv_status novakv_debug_set_scan_ctas(novakv_ctx* ctx, int n_ctas);

/*
 * Value-accumulation variant of the decode scan kernel: 1 (default) runs sum_j p_j * codeword_j on
 * tensor cores (fp16 weights and codewords, fp32 accumulation); 0 keeps it on CUDA cores in fp32.
 * Both are held to the same output tolerance; the benchmark reports both.
 */
novakv_status novakv_debug_set_value_path(novakv_ctx* ctx, int path);

/*
 * Work split of the index scan.  The scan kernel walks all (sequence, KV head) pairs page by page and
 * cuts the walk into one contiguous piece per CTA.  Each pair a CTA touches costs it a fixed set-up (the
 * per-query score table), so the cut is even not in pages but in pages + `pages` per pair touched: a CTA
 * that has to set up several pairs gets fewer pages.  `pages` = 0 gives the even split in pages; the
 * default is 24.  Results do not depend on it beyond binary32 rounding (it only moves split points).
 */
novakv_status novakv_debug_set_segment_weight(novakv_ctx* ctx, int pages);

/*
 * Cross-split merge (App. B "Decoding kernel and read path": stage 2 combines the per-split partials).
 * on = 0 (default): a separate merge kernel follows the scan.  on = 1: without a sink logit and without a
 * BF16 band the scan kernel performs the merge itself - the CTA that writes the last partial of a
 * (sequence, KV head) pair combines the pair's partials and applies the inverse value transform; an arrival
 * counter per pair decides, nothing waits.  Results agree within binary32 rounding.  (Measured on B200 the
 * fused form saves a launch but puts the merge on the critical path of the last CTA of every pair; it is not
 * faster at any benchmark shape, hence not the default.)
 */
novakv_status novakv_debug_set_fused_merge(novakv_ctx* ctx, int on);

/* Kernels this library launched since the context was created (all kinds). */
long novakv_launch_count(const novakv_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* NOVAKV_H */
