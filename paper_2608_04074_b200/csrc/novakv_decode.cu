// Read path: decode-step attention straight from the packed index cache.
//
//   prepare  : q' = sm_scale*log2(e) * q rk_inv_t  per head, and a prefix sum of page counts (the
//              work list of the scan kernel: one unit = one 64-token page of one (sequence, KV head)).
//   stage 1  : persistent scan kernel, one CTA per SM.  Each CTA takes a contiguous range of the
//              global page sequence, so that consecutive pages mostly belong to the same
//              (sequence, KV head) and reuse its score table.  Per (sequence, KV head) segment:
//                - score table LUT[code][l][h] = <q'_h[4l..4l+3], cb_k[l][code] - centre_l> in shared memory,
//                  all heads of the KV head side by side in one entry.  The first K32 groups, which carry
//                  the high-variance coordinates and hence the large entries, are kept in binary32; the
//                  others (head dimension 128 only) in binary16,
//                - every warp streams its own 32-token tiles with coalesced 128-bit loads straight into
//                  registers, the next tile's loads in flight while the current tile is consumed (the
//                  cache layout is such that each lane's bytes are exactly the ones it consumes),
//                - key side: lane <-> token, L table lookups summed in registers (no cross-lane
//                  reduction): binary32 adds for the binary32 entries, short binary16 chains, each
//                  flushed into the binary32 sum, for the others,
//                - online softmax per 32-token tile with a lazily updated running maximum,
//                - value side: sum_j p_j * value-codeword_j in the value-transform domain, a dense
//                  [heads x tokens] x [tokens x d] contraction, run on tensor cores (mma.sync, binary16
//                  operands, binary32 accumulators) or, as the selectable alternative, on CUDA cores in
//                  binary32; value codewords are 7-bit grid indices (4 bytes per codeword) that expand to
//                  binary16 with one byte permutation per pair,
//                - the warps' partial (m, l, acc) are merged and written once per segment.
//   merge    : exact log-sum-exp merge of the partials of every (sequence, KV head), then the inverse
//              value transform o = o' rv^T + v_mean, once per head.
//
// Shared-memory gathers are laid out against bank conflicts: byte j of a token's key bytes holds group
// j ^ (token % 8) (j ^ (token % 16) for j >= 16), so that at every step the lanes of a quarter warp read 8
// different 16-byte columns of a binary32 table row and the lanes of a half warp 16 different 8-byte
// columns of a binary16 row (steps 8..15 meet only 8 groups: those groups are stored a second time in the
// unused first columns of the row and the upper half of a half warp reads the copy); on the value
// side the 32 lanes of a warp read 32 different 4-byte slots, because the lane columns fc = 0,1 and fc = 2,3
// use two copies of the value codebook whose slots are rotated by 16, and odd columns take the group
// blocks in swapped order (the cache stores their bytes in that order, and the byte permutation that widens a
// codeword for the tensor core picks it from the swapped register).
// The kernel contains no spin wait.
#include <math_constants.h>
#ifdef NOVAKV_TIMING
#include <cstdio>
#endif

#include "novakv_internal.cuh"

namespace {

#ifndef NOVAKV_NCW
#define NOVAKV_NCW 16
#endif
#ifndef NOVAKV_CHAIN
#define NOVAKV_CHAIN 4        // table lookups summed in binary16 before a flush into the binary32 logit
#endif
#ifndef NOVAKV_KSC_CHAIN
#define NOVAKV_KSC_CHAIN 2
#endif
#ifndef NOVAKV_WINDOW
#define NOVAKV_WINDOW 8       // tiles whose tensor-core sums are accumulated before the centre of the value grid is removed
#endif
constexpr int NCW = NOVAKV_NCW;               // warps of the scan kernel
constexpr int S1_THREADS = NCW * 32;
constexpr int T16_BYTES = 65536;              // binary16 table: 256 codes x 256-byte rows
constexpr int T16_ROW = 256;
constexpr int VCB_COPY_BYTES = 32768;         // 256 codes x 32 slots x 4 bytes
constexpr int VCB_ROW = 128;
constexpr int S1_SMEM_BYTES = 229376;         // dynamic shared memory requested (224 KB; the CTA also has a few static words)
constexpr float M_INIT = -1.0e30f;
#ifndef NOVAKV_M_SLACK
#define NOVAKV_M_SLACK 4
#endif
constexpr float M_SLACK = (float)NOVAKV_M_SLACK;   // headroom (bits) a running maximum gets when it moves
constexpr int MAX_SCAN_CTAS = 255;            // scan CTAs (one per SM) the boundary table has room for
constexpr int PFX_CAP = 511;                  // batches up to this size keep their page / cost prefixes in shared memory

// VM selects the value side: true = tensor cores (mma.sync m16n8k16, fp16 weights and codewords,
// fp32 accumulators), false = CUDA cores (fp32 FMA).
template <int D, int HG, bool VM>
struct S1 {
    static constexpr int L = D / NOVAKV_G;
    static constexpr int NGB = L / 8;                         // group blocks of 8 groups (value side)
    static constexpr int KPL = L / 16;                        // 16-byte planes of a key tile: 2 or 1
    static constexpr int HSETS = HG <= 4 ? 1 : 2;             // sets of 4 heads
    static constexpr int HPAD = HSETS * 4;
    // Score table.  Groups 0 .. K32-1 (the equal-volume dealing puts the coordinates of largest variance there)
    // have binary32 entries, 16 bytes per head set: T32[hs][code][K32][4 heads].  The other groups have
    // binary16 entries, 8 bytes: T16[code][32 columns][4 heads], rows of 256 bytes (only for d = 128, where
    // Hq/Hkv <= 4).  For d = 64 every group is binary32.
    static constexpr int K32 = D == 128 ? 8 : L;
    static constexpr bool HAS16 = K32 < L;
    static_assert(!HAS16 || HSETS == 1, "binary16 entries hold one head set");
    static constexpr int ROW32 = K32 * 16;
    static constexpr int PLANE32 = 256 * ROW32;
    static constexpr int T32_BYTES = HSETS * PLANE32;
    static constexpr int TILE_BYTES = 32 * L;                 // index bytes of a 32-token tile, K or V
    // per-warp staging of the softmax weights of one 32-token tile
    //   VM: fp16 [HPAD][4 k-slot pairs][8 tokens]        otherwise: fp32 [32 tokens][HPAD]
    static constexpr int P_WARP_BYTES = VM ? HPAD * 64 : 32 * HPAD * 4;
    static constexpr int P_BYTES = NCW * P_WARP_BYTES;
    // Shared-memory map.  Below the binary16 table: T32, the weight staging, q' of the pair.  The binary16 table
    // sits at the first 64 KB boundary of the shared address window that leaves that much room (a row then
    // starts at an address whose low 16 bits are code * 256, so that one byte permutation builds a gather
    // address); without a binary16 table nothing needs aligning.  The two copies of the value codebook follow.
    static constexpr int OFFB_T32 = 0;
    static constexpr int OFFB_P = OFFB_T32 + T32_BYTES;
    static constexpr int OFFB_Q = OFFB_P + P_BYTES;                     // fp32 [HPAD][D]
    static constexpr int OFFB_BND = OFFB_Q + HPAD * D * 4;              // long [MAX_SCAN_CTAS + 1]: first unit of every CTA
    static constexpr int OFFB_PFX = OFFB_BND + (MAX_SCAN_CTAS + 1) * 8; // int [2][PFX_CAP + 1]: page and cost prefix of small batches
    static constexpr int BELOW_BYTES = OFFB_PFX + 2 * (PFX_CAP + 1) * 4;
    // merge buffer (aliases the larger table once a segment's scan is done)
    static constexpr int MROW = D + 4;                                  // floats per (warp, head) row of the merge buffer: 16 bytes of padding
                                                                        // keep the four head rows a warp writes at once on different banks
    static constexpr int MERGE_ACC_BYTES = NCW * HPAD * MROW * 4;
    static_assert(MERGE_ACC_BYTES + NCW * HPAD * 16 <= (HAS16 ? T16_BYTES : T32_BYTES), "merge buffer must fit in a table");
    static_assert(BELOW_BYTES + (HAS16 ? T16_BYTES : 0) + 2 * VCB_COPY_BYTES <= S1_SMEM_BYTES, "shared memory budget (before alignment)");
    static_assert(S1_THREADS % L == 0, "table build mapping");
};

__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ int clamp_len(int len, int max_pages) {
    const int cap = max_pages * NOVAKV_PAGE_TOKENS;
    return len < 0 ? 0 : (len > cap ? cap : len);
}

// ------------------------------------------------------------------------------------------------
// prepare: query transform + page prefix
// ------------------------------------------------------------------------------------------------
// One block per (sequence, KV head): the Hg queries of the head share every load of rk_inv_t.
// 512 threads = D columns x (512/D) row parts; each thread's loads are independent and all in flight.
template <int D, int HG>
__global__ void __launch_bounds__(512)
novakv_prepare_kernel(const __nv_bfloat16* __restrict__ q, const float* __restrict__ rk_inv_t,
                      const int32_t* __restrict__ seq_lens, int batch, int n_q_heads, int n_kv_heads,
                      int max_pages_per_seq, float scale_log2, float* __restrict__ qp,
                      int32_t* __restrict__ page_prefix, uint32_t* __restrict__ dev_status,
                      const float* __restrict__ k_mean /* [Hkv][D] */, float* __restrict__ qk_off /* [batch][Hq] or null */,
                      int32_t* __restrict__ cost_prefix /* [batch + 1] */, int seg_weight,
                      const float* __restrict__ k_center /* [Hkv][D], transform domain */, float* __restrict__ qc /* [batch][Hq] or null */,
                      int32_t* __restrict__ pair_count /* [Hkv * batch] arrival counters of the fused merge, or null */,
                      void* __restrict__ out_fused /* outputs, when the scan kernel itself merges */, int out_is_fp32) {
    const int blk = blockIdx.x;
#ifdef NOVAKV_TIMING
    unsigned long long g_p0, g_p1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g_p0));
#endif
    constexpr int PARTS = 512 / D, ROWS = D / PARTS;
    const int b = blk / n_kv_heads, kvh = blk - b * n_kv_heads;
    const int c = threadIdx.x % D, part = threadIdx.x / D;
    // The query transform depends on nothing the preceding kernel of the stream (normally the append of this
    // step's tokens) writes: queries are produced before that kernel started, the transform is a constant.  So
    // the blocks that transform queries never wait on the grid dependency: they run beside the preceding
    // kernel.  Only the block that forms the page prefix (it reads seq_lens, which an append updates) waits;
    // since a grid completes only when all its blocks have, the scan kernel's own wait still covers both.
    float rv[ROWS];
    if (blk < batch * n_kv_heads) {
        const float* R = rk_inv_t + (size_t)kvh * D * D + (size_t)part * ROWS * D + c;
#pragma unroll
        for (int r = 0; r < ROWS; ++r) rv[r] = R[(size_t)r * D];
    }
    if (blk == batch * n_kv_heads) {
        novakv_grid_dependency_wait();
        // exclusive prefix over sequences of their page counts; small, done by one warp.  Beside it the same
        // prefix in "cost" units, in which every non-empty sequence weighs seg_weight pages more: the scan
        // kernel splits the walk evenly in cost, so that a CTA that has to set up several (sequence, KV head)
        // segments gets fewer pages.
        if (threadIdx.x < 32) {
            int carry = 0, carry_ne = 0;
            for (int b0 = 0; b0 < batch; b0 += 32) {
                const int b = b0 + threadIdx.x;
                int v = 0;
                if (b < batch) {
                    const int raw = seq_lens[b];
                    const int len = clamp_len(raw, max_pages_per_seq);
                    if (raw != len) atomicOr(dev_status, NOVAKV_DEV_BAD_LENGTH);
                    v = (len + NOVAKV_PAGE_TOKENS - 1) / NOVAKV_PAGE_TOKENS;
                }
                const int ne = v > 0 ? 1 : 0;
                int incl = v, incl_ne = ne;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t = __shfl_up_sync(0xffffffffu, incl, o);
                    const int tn = __shfl_up_sync(0xffffffffu, incl_ne, o);
                    if ((int)threadIdx.x >= o) { incl += t; incl_ne += tn; }
                }
                if (b < batch) {
                    page_prefix[b] = carry + incl - v;
                    cost_prefix[b] = carry + incl - v + seg_weight * (carry_ne + incl_ne - ne);
                }
                // no scan CTA ever visits an empty sequence: with the merge fused into the scan its zeros are written here
                if (out_fused != nullptr) {
                    const unsigned empties = __ballot_sync(0xffffffffu, b < batch && v == 0);
                    for (unsigned m = empties; m; m &= m - 1) {
                        const size_t row = (size_t)(b0 + __ffs(m) - 1) * n_q_heads * D;
                        for (int i = threadIdx.x; i < n_q_heads * D; i += 32) {
                            if (out_is_fp32) reinterpret_cast<float*>(out_fused)[row + i] = 0.f;
                            else reinterpret_cast<__nv_bfloat16*>(out_fused)[row + i] = __float2bfloat16_rn(0.f);
                        }
                    }
                }
                carry += __shfl_sync(0xffffffffu, incl, 31);
                carry_ne += __shfl_sync(0xffffffffu, incl_ne, 31);
            }
            if (threadIdx.x == 0) { page_prefix[batch] = carry; cost_prefix[batch] = carry + seg_weight * carry_ne; }
        }
#ifdef NOVAKV_TIMING
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g_p1));
        if (threadIdx.x == 0) printf("prepare prefix block | ns start %llu end %llu\n", g_p0, g_p1);
#endif
        return;
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (pair_count != nullptr && threadIdx.x == 0) pair_count[kvh * batch + b] = 0;
    __shared__ float q_s[HG][D];
    __shared__ float red_s[PARTS][HG][D];
    for (int i = threadIdx.x; i < HG * D; i += 512)
        q_s[i / D][i % D] = __bfloat162float(q[((size_t)b * n_q_heads + kvh * HG) * D + i]);
    __syncthreads();
    float acc[HG];
#pragma unroll
    for (int h = 0; h < HG; ++h) acc[h] = 0.f;
#pragma unroll
    for (int r = 0; r < ROWS; ++r)
#pragma unroll
        for (int h = 0; h < HG; ++h) acc[h] = fmaf(q_s[h][part * ROWS + r], rv[r], acc[h]);
#pragma unroll
    for (int h = 0; h < HG; ++h) red_s[part][h][c] = acc[h];
    __syncthreads();
    for (int i = threadIdx.x; i < HG * D; i += 512) {
        const int h = i / D, cc = i % D;
        float v = 0.f;
#pragma unroll
        for (int p = 0; p < PARTS; ++p) v += red_s[p][h][cc];
        v *= scale_log2;
        qp[((size_t)b * n_q_heads + kvh * HG + h) * D + cc] = v;
        if (qc != nullptr) red_s[0][h][cc] = v * k_center[(size_t)kvh * D + cc];       // (each thread rewrites only what it read)
    }
    // the constant the read path drops from every logit of a query, q . k_mean * sm_scale (base-2 units):
    // only a learned sink logit and the BF16 band need it (they must be shifted by the same amount)
    if (qk_off != nullptr && (threadIdx.x >> 5) < HG) {
        const int h = threadIdx.x >> 5, lane = threadIdx.x & 31;
        float acc = 0.f;
        for (int i = lane; i < D; i += 32) acc = fmaf(q_s[h][i], k_mean[(size_t)kvh * D + i], acc);
        acc = warp_sum_f(acc);
        // (the merge kernel of a preceding decode call on this workspace reads qk_off: its grid must have completed)
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (lane == 0) qk_off[(size_t)b * n_q_heads + kvh * HG + h] = acc * scale_log2;
    }
    // scaled key format: the table is built from centred codewords, and the centre's share <q', centre> of
    // every logit is added back before the per-token scale multiplies it
    if (qc != nullptr) {
        __syncthreads();
        if ((threadIdx.x >> 5) < HG) {
            const int h = threadIdx.x >> 5, lane = threadIdx.x & 31;
            float acc = 0.f;
            for (int i = lane; i < D; i += 32) acc += red_s[0][h][i];
            acc = warp_sum_f(acc);
            if (lane == 0) qc[(size_t)b * n_q_heads + kvh * HG + h] = acc;
        }
    }
#ifdef NOVAKV_TIMING
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g_p1));
    if (threadIdx.x == 0 && (blk == 0 || blk == batch * n_kv_heads - 1))
        printf("prepare block %d | ns start %llu end %llu\n", blk, g_p0, g_p1);
#endif
}

// ------------------------------------------------------------------------------------------------
// stage 1 helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint2 lds_u64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds_u128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
// Byte permutation with the full selector of the instruction: bit 3 of a selector nibble replaces the chosen
// byte by eight copies of its top bit (the intrinsic __byte_perm documents only the low three bits).
__device__ __forceinline__ uint32_t prmt_rep(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1,%2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0,%1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// packed binary32 pairs (two IEEE operations per instruction)
__device__ __forceinline__ void fadd2(uint64_t& d, uint64_t a) {
    asm("add.rn.f32x2 %0, %0, %1;" : "+l"(d) : "l"(a));
}
__device__ __forceinline__ void ffma2(uint64_t& d, uint64_t a, uint64_t b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}
__device__ __forceinline__ void fmul2(uint64_t& d, uint64_t a) {
    asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(d) : "l"(a));
}
// packed binary16 pairs
__device__ __forceinline__ uint32_t hadd2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("add.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// lo += low half of h, hi += high half of h (binary16 widened exactly, binary32 addition)
__device__ __forceinline__ void flush_h2(uint32_t h, float& lo, float& hi) {
    asm("{\n\t.reg .b16 l, u;\n\tmov.b32 {l, u}, %2;\n\tadd.rn.f32.f16 %0, l, %0;\n\tadd.rn.f32.f16 %1, u, %1;\n\t}"
        : "+f"(lo), "+f"(hi) : "r"(h));
}
__device__ __forceinline__ uint32_t pack_h2(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float warp_max(float v) {
    int i = __float_as_int(v);
    i ^= (i >> 31) & 0x7fffffff;               // order-preserving map to signed integers
    i = __reduce_max_sync(0xffffffffu, i);
    i ^= (i >> 31) & 0x7fffffff;
    return __int_as_float(i);
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct Segment {
    int b, kvh, pg0, npg, len;
};

// Locate the (KV head, sequence, page) of global page unit u.  Units are ordered KV-head-major:
// u = kvh * P + page_prefix[b] + page, with P = page_prefix[batch] the pages of all sequences, so that
// consecutive segments of a CTA share the KV head (and its value codebook).  page_prefix is exclusive,
// length batch + 1.  Cooperative: every thread tests one sequence (all loads independent, one memory
// latency), the owner publishes (b, length) through shared memory.  Contains a __syncthreads().
__device__ __forceinline__ Segment locate(const int32_t* __restrict__ page_prefix, const int32_t* __restrict__ seq_lens,
                                          int batch, int max_pages, long u, long u_end, int* s_found) {
    const long P = page_prefix[batch];
    Segment s;
    s.kvh = (int)(u / P);
    const long r = u - (long)s.kvh * P;
    for (int t = threadIdx.x; t < batch; t += S1_THREADS) {
        const int lo = page_prefix[t], hi = page_prefix[t + 1], len = seq_lens[t];
        if ((long)lo <= r && r < (long)hi) { s_found[0] = t; s_found[1] = clamp_len(len, max_pages); s_found[2] = lo; }
    }
    __syncthreads();
    s.b = s_found[0];
    s.len = s_found[1];
    const int pages_b = (s.len + NOVAKV_PAGE_TOKENS - 1) / NOVAKV_PAGE_TOKENS;
    s.pg0 = (int)(r - s_found[2]);
    const long left = u_end - u;
    s.npg = (int)(left < (long)(pages_b - s.pg0) ? left : (long)(pages_b - s.pg0));
    return s;
}

// ------------------------------------------------------------------------------------------------
// stage 1: persistent index scan
// ------------------------------------------------------------------------------------------------
// Streaming 128-/64-bit loads of index bytes: read once, keep them out of L1.
__device__ __forceinline__ uint4 ldg_stream_128(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ldg_stream_64(const void* p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

// Value codebook of a KV head (32 KB image, uint8 [256 codes][32 slots][4], slot = group) -> two copies in
// shared memory, copy c holding group g in slot (g + 16 c) % 32, without registers: asynchronous 16-byte
// copies that land while the caller does other work (segment lookup, page ids, table build);
// async_copies_wait() before the barrier that publishes the copies.  A 16-byte chunk holds 4 slots, so the
// rotation by 16 slots moves whole chunks.  INTERLEAVED: the two copies share 256-byte rows
// [code][copy][32 slots] (a row then starts at code * 256 of a 64 KB block); otherwise copy 1 follows copy 0.
template <bool INTERLEAVED>
__device__ __forceinline__ void stage_value_codebook_async(unsigned char* vcb, const uint8_t* __restrict__ src_g) {
    const uint32_t d0 = smem_u32(vcb);
    for (int i = threadIdx.x; i < VCB_COPY_BYTES / 16; i += S1_THREADS) {
        const int row = i >> 3, ch = i & 7;
        const uint8_t* src = src_g + (size_t)i * 16;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            const uint32_t dst = d0 + (INTERLEAVED ? row * (2 * VCB_ROW) + c * VCB_ROW : c * VCB_COPY_BYTES + row * VCB_ROW) +
                                 ((ch + 4 * c) & 7) * 16;
            asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}
__device__ __forceinline__ void async_copies_wait() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// The table build is kept out of line so that its load batches do not disturb the register allocation of
// the scan loop.  Entry (code, l, h) = <q'_h segment of group l, centred key codeword (l, code)>, heads beyond
// HG zero: binary32 in T32 for l < K32, binary16 in T16 otherwise.
template <int D, int HG, bool VM>
__device__ __noinline__ void build_score_table(unsigned char* t32, unsigned char* t16,
                                               const float* __restrict__ cb_k_lut /* [256][L][4] of the KV head */,
                                               const float* q_s /* shared: q' of the pair, [HPAD][D] */) {
    using C = S1<D, HG, VM>;
    constexpr int L = C::L, HPAD = C::HPAD, HSETS = C::HSETS, K32 = C::K32;
    if constexpr (C::HAS16) {
        // Hybrid table: whole warps take one kind of entry, so that no warp runs both store paths.  Threads
        // 0 .. 16 K32 - 1 build the binary32 part (group = t % K32, 16 codes per pass), the others the binary16
        // part (group = K32 + t' % (L - K32), 16 codes per pass); 16 passes either way.
        static_assert(K32 == 8 && L == 32 && S1_THREADS == 512 && HPAD == 4, "work split of the hybrid table build");
        constexpr int T32_THREADS = 16 * K32;                   // 128 = 4 warps
        constexpr int BATCH = 8;
        const bool is32 = threadIdx.x < T32_THREADS;
        const int tl = is32 ? threadIdx.x : threadIdx.x - T32_THREADS;
        const int g = is32 ? tl % K32 : K32 + tl % (L - K32);
        const int code0 = is32 ? tl / K32 : tl / (L - K32);
        float4 qs[HPAD];
#pragma unroll
        for (int h = 0; h < HPAD; ++h) qs[h] = *reinterpret_cast<const float4*>(q_s + h * D + g * 4);
        const float4* cbk = reinterpret_cast<const float4*>(cb_k_lut) + g;
        const uint32_t a32 = smem_u32(t32) + g * 16, a16 = smem_u32(t16) + g * 8;
#pragma unroll 1
        for (int it0 = 0; it0 < 16; it0 += BATCH) {
            float4 cw[BATCH];
#pragma unroll
            for (int u = 0; u < BATCH; ++u) cw[u] = cbk[(size_t)(code0 + (it0 + u) * 16) * L];
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                const int code = code0 + (it0 + u) * 16;
                float o[HPAD];
#pragma unroll
                for (int h = 0; h < HPAD; ++h)
                    o[h] = fmaf(qs[h].w, cw[u].w, fmaf(qs[h].z, cw[u].z, fmaf(qs[h].y, cw[u].y, qs[h].x * cw[u].x)));
                if (is32) {
                    asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(a32 + code * C::ROW32),
                                 "f"(o[0]), "f"(o[1]), "f"(o[2]), "f"(o[3]) : "memory");
                } else {
                    // (a table entry beyond the binary16 range would be a logit share of 2^16 bits; clamped, never inf)
                    const uint32_t e0 = pack_h2(fminf(fmaxf(o[0], -60000.f), 60000.f), fminf(fmaxf(o[1], -60000.f), 60000.f));
                    const uint32_t e1 = pack_h2(fminf(fmaxf(o[2], -60000.f), 60000.f), fminf(fmaxf(o[3], -60000.f), 60000.f));
                    asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(a16 + code * T16_ROW), "r"(e0), "r"(e1) : "memory");
                    // groups 8..15 a second time in columns 0..7: the 16 lanes of a half warp then read 16 different columns
                    if (g < 16) asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(a16 + code * T16_ROW - 64), "r"(e0), "r"(e1) : "memory");
                }
            }
        }
        return;
    }
    constexpr int CSTEP = S1_THREADS / L;                       // codes per pass of the CTA
    constexpr int NIT = (256 + CSTEP - 1) / CSTEP;
    constexpr int BATCH = 8;                                    // loads in flight per thread
    const int g = threadIdx.x % L, code0 = threadIdx.x / L;
    float4 qs[HPAD];
#pragma unroll
    for (int h = 0; h < HPAD; ++h) qs[h] = *reinterpret_cast<const float4*>(q_s + h * D + g * 4);
    const float4* cbk = reinterpret_cast<const float4*>(cb_k_lut);
#pragma unroll 1
    for (int it0 = 0; it0 < NIT; it0 += BATCH) {
        float4 cw[BATCH];
#pragma unroll
        for (int u = 0; u < BATCH; ++u) {
            const int code = code0 + (it0 + u) * CSTEP;
            if (it0 + u < NIT && code < 256) cw[u] = cbk[(size_t)code * L + g];
        }
#pragma unroll
        for (int u = 0; u < BATCH; ++u) {
            const int code = code0 + (it0 + u) * CSTEP;
            if (it0 + u < NIT && code < 256) {
                float o[HPAD];
#pragma unroll
                for (int h = 0; h < HPAD; ++h)
                    o[h] = fmaf(qs[h].w, cw[u].w, fmaf(qs[h].z, cw[u].z, fmaf(qs[h].y, cw[u].y, qs[h].x * cw[u].x)));
                if (g < K32) {
#pragma unroll
                    for (int hs = 0; hs < HSETS; ++hs)
                        *reinterpret_cast<float4*>(t32 + hs * C::PLANE32 + code * C::ROW32 + g * 16) =
                            make_float4(o[hs * 4], o[hs * 4 + 1], o[hs * 4 + 2], o[hs * 4 + 3]);
                } else if (C::HAS16) {
                    // (a table entry beyond the binary16 range would be a logit share of 2^16 bits; clamped, never inf)
                    const uint2 e = make_uint2(pack_h2(fminf(fmaxf(o[0], -60000.f), 60000.f), fminf(fmaxf(o[1], -60000.f), 60000.f)),
                                               pack_h2(fminf(fmaxf(o[2], -60000.f), 60000.f), fminf(fmaxf(o[3], -60000.f), 60000.f)));
                    *reinterpret_cast<uint2*>(t16 + code * T16_ROW + g * 8) = e;
                    // groups 8..15 a second time in columns 0..7: the 16 lanes of a half warp then read 16 different columns
                    if (K32 == 8 && g < 16) *reinterpret_cast<uint2*>(t16 + code * T16_ROW + (g - 8) * 8) = e;
                }
            }
        }
    }
}

// Index bytes of one 32-token tile as one lane holds them.
//   kw: this lane's token (lane = token within the tile), L bytes: byte j holds the code of group
//       j ^ (lane % 8) for j < 16 and j ^ (lane % 16) for j >= 16.
//   vw: per 16-token block, the codes of this lane's MMA coordinates (fr = lane/4, fc = lane%4):
//       word gb holds, for the four tokens 4u + fc of the block (byte u), the code of group 8 gb + fr.
template <int L>
struct TileRegs {
    uint32_t kw[L / 4];
    uint32_t vw[2][L / 8];
    uint32_t ks;          // this lane's token: bfloat16 key scale in the high half (a binary32 bit pattern), if used
    uint32_t vm;          // this lane's token: bfloat16 value scale (low half) and zero-point (high half), if used
};

// First unit of scan CTA c of G (c = G gives the end of the walk).  The walk is cut evenly in cost units,
// cost = pages + seg_weight per (sequence, KV head) pair: cost point t lies in the pair whose cost interval
// contains it and maps to unit  start + clamp(t - cost_start - seg_weight, 0, pages)  (the first seg_weight cost
// units of a pair stand for setting up its score table).  seg_weight = 0 is the even split in pages.
__device__ __forceinline__ long scan_boundary(int c, int G, const int32_t* __restrict__ page_prefix,
                                              const int32_t* __restrict__ cost_prefix, int batch, int n_kv_heads, int seg_weight) {
    const long P = page_prefix[batch], U = P * n_kv_heads;
    if (seg_weight == 0) return ((long)c * U) / G;
    const long cper = cost_prefix[batch], T = cper * n_kv_heads;
    const long t = ((long)c * T) / G;
    if (cper <= 0 || t >= T) return U;
    const long kv = t / cper, rem = t - kv * cper;
    int lo = 0, hi = batch - 1;                   // the last sequence whose cost interval starts at or before rem
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if ((long)cost_prefix[mid] <= rem) lo = mid; else hi = mid - 1;
    }
    const long p0 = page_prefix[lo], pg = page_prefix[lo + 1] - p0;
    return kv * P + p0 + min(max(rem - cost_prefix[lo] - seg_weight, 0l), pg);
}

// Merge of one (sequence, KV head) pair inside the scan kernel, run by the CTA that wrote the pair's last
// partial: exact log-sum-exp combination of the partials of the CTAs first .. last (those with an empty
// range skipped), normalisation, inverse value transform o = o' rv^T + v_mean.  scratch: shared memory,
// (1 + S1_THREADS / D) * HG * D floats.  Partials of other CTAs are read past the L1 (they were written by
// other SMs; the arrival counter orders the accesses).
template <int D, int HG>
__device__ __noinline__ void fused_merge(float* scratch, const float* part_ml, const float* part_acc, int pair, int first,
                                         int last, const long* s_bnd, const float* __restrict__ rv_t,
                                         const float* __restrict__ v_mean, int kvh, void* __restrict__ out, int out_is_fp32,
                                         size_t out_row /* (b * Hq + kvh * HG) * D */) {
    constexpr int PARTS = S1_THREADS / D, COLS = D / PARTS;
    float* o_s = scratch;                         // [HG][D]
    float* red_s = scratch + HG * D;              // [PARTS][HG][D]
    for (int i = threadIdx.x; i < HG * D; i += S1_THREADS) {
        const int h = i / D, c = i - h * D;
        float M = M_INIT;
        for (int cta = first; cta <= last; ++cta)
            if (s_bnd[cta] < s_bnd[cta + 1]) M = fmaxf(M, __ldcg(part_ml + (((size_t)pair + cta) * HG + h) * 2));
        float a = 0.f, lsum = 0.f;
        for (int cta = first; cta <= last; ++cta) {
            if (s_bnd[cta] >= s_bnd[cta + 1]) continue;
            const size_t pidx = (size_t)pair + cta;
            const float sc = ex2(__ldcg(part_ml + (pidx * HG + h) * 2) - M);
            a = fmaf(sc, __ldcg(part_acc + (pidx * HG + h) * D + c), a);
            lsum = fmaf(sc, __ldcg(part_ml + (pidx * HG + h) * 2 + 1), lsum);
        }
        o_s[i] = lsum > 0.f ? a / lsum : 0.f;
    }
    __syncthreads();
    {
        const int r = threadIdx.x % D, part = threadIdx.x / D;
        const float* R = rv_t + (size_t)kvh * D * D + (size_t)part * COLS * D + r;      // rv_t[c][r] = R_V[r][c]
        float acc[HG];
#pragma unroll
        for (int h = 0; h < HG; ++h) acc[h] = 0.f;
#pragma unroll 8
        for (int c = 0; c < COLS; ++c) {
            const float rv = R[(size_t)c * D];
#pragma unroll
            for (int h = 0; h < HG; ++h) acc[h] = fmaf(o_s[h * D + part * COLS + c], rv, acc[h]);
        }
#pragma unroll
        for (int h = 0; h < HG; ++h) red_s[(part * HG + h) * D + r] = acc[h];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < HG * D; i += S1_THREADS) {
        const int h = i / D, r = i - h * D;
        float o = v_mean[(size_t)kvh * D + r];
#pragma unroll
        for (int p = 0; p < PARTS; ++p) o += red_s[(p * HG + h) * D + r];
        if (out_is_fp32) reinterpret_cast<float*>(out)[out_row + i] = o;
        else reinterpret_cast<__nv_bfloat16*>(out)[out_row + i] = __float2bfloat16_rn(o);
    }
}

// KSC: the key format carries a per-token bfloat16 scale (k_scales [n_pages][Hkv][64]); the logits of a
// token are multiplied by it once, after the table lookups are summed (and the centre's share added back).
// VSQ: scalar INT2 values with a per-token bfloat16 scale and zero-point (v_meta [n_pages][Hkv][64][2]).
// A byte of four 2-bit codes indexes the product codebook {0,1,2,3}^4, so the value side is the same gather
// with that fixed table as the value-codebook image; the weight of a token's codes is p * scale and the
// zero-points enter through one extra running sum per head, sum_j p_j zero_j, added to every coefficient
// in the epilogue.
//
// Numerics of the tensor-core value side.  A softmax weight enters the product as the binary16 number
// w = fp16(2^15 p) (p <= 1 relative to the running maximum, so w <= 2^15; weights down to 2^-39 stay
// non-zero), and the same rounded w is what the normaliser sums: the result is an exact softmax of slightly
// perturbed logits.  A value codeword is four 7-bit grid indices u (bytes with the top bit clear); the byte
// permutation that widens them pairs every byte with its replicated top bit, i.e. with a zero byte: the
// binary16 numbers u 2^-24 (subnormal, exact; the tensor core multiplies them exactly).  The same permutation
// picks the bytes from one of two registers by lane, which undoes the block swap of the odd lane columns.
// Every NOVAKV_WINDOW tiles, and before any rescaling, the grid centre is removed with the weight sum of
// the same tokens (every lane adds up the rounded weights of its own tokens; a shuffle reduction per window
// gives each lane column the sum of its head): acc -= 64 2^-24 sum_j w_j leaves 2^-24 sum_j w_j (u_j - 64),
// so that the long-running sums stay centred.  (An all-ones operand on the tensor core gave the same sums at
// four more matrix instructions per tile, which cost more issue time than the shuffles.)
template <int D, int HG, bool VM, bool KSC, bool VSQ>
__global__ void __launch_bounds__(S1_THREADS, 1)
novakv_decode_stage1_kernel(const float* __restrict__ qp, const float* __restrict__ cb_k_lut,
                            const uint8_t* __restrict__ cb_v_img, const float* __restrict__ v_scale,
                            const float* __restrict__ v_off, const uint8_t* __restrict__ k_pages,
                            const uint8_t* __restrict__ v_pages, const __nv_bfloat16* __restrict__ k_scales,
                            const __nv_bfloat16* __restrict__ v_meta, int n_pages,
                            const int32_t* __restrict__ page_table, int max_pages_per_seq,
                            const int32_t* __restrict__ seq_lens, const int32_t* __restrict__ page_prefix,
                            int batch, int n_q_heads, int n_kv_heads, float* __restrict__ part_ml,
                            float* __restrict__ part_acc, uint32_t* __restrict__ dev_status, int pt_stride,
                            const int32_t* __restrict__ cost_prefix, int seg_weight, long* __restrict__ cta_range,
                            const float* __restrict__ qc, int vcb_per_head,
                            int32_t* __restrict__ pair_count, const float* __restrict__ rv_t,
                            const float* __restrict__ v_mean, void* __restrict__ out_fused, int out_is_fp32) {
    // out_fused != null: the CTA that writes the last partial of a (sequence, KV head) pair also merges the pair's
    // partials and applies the inverse value transform (no merge kernel follows); pair_count holds one arrival
    // counter per pair, zero on entry and reset to zero by the merging CTA.  Nothing waits on another CTA.
    // page_table points at the first column that is scanned; rows are pt_stride entries apart and
    // max_pages_per_seq bounds the pages of a row that may be read from there
    using C = S1<D, HG, VM>;
    constexpr int L = C::L, HPAD = C::HPAD, HSETS = C::HSETS, NGB = C::NGB, KPL = C::KPL, K32 = C::K32;
    constexpr bool HAS16 = C::HAS16;
    constexpr int TILE_BYTES = C::TILE_BYTES, PAGE_BYTES = 2 * TILE_BYTES;
    constexpr float SH = VM ? 15.f : 0.f;                     // weights are scaled by 2^SH before the binary16 rounding
    constexpr float U_UNIT = 5.9604644775390625e-08f;         // 2^-24: a grid index u enters a product as the binary16 subnormal u 2^-24
    constexpr float CEN = VSQ ? 0.f : 64.f * U_UNIT;          // what one unit of weight adds to a tensor-core sum beyond u - centre
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ int s_found[4];
    __shared__ int s_arrived, s_first, s_last;
    // ---- shared-memory map (see S1)
    const uint32_t s_base = smem_u32(smem);
    const uint32_t t16_abs = HAS16 ? ((s_base + C::BELOW_BYTES + 65535u) & ~65535u) : s_base + C::BELOW_BYTES;
    const uint32_t pad = t16_abs - s_base;
    if (pad + (HAS16 ? T16_BYTES : 0) + 2 * VCB_COPY_BYTES > (uint32_t)S1_SMEM_BYTES || (s_base & 255u) != 0u) {
        // cannot happen with the shared address window of this architecture; reported, never trapped
        if (threadIdx.x == 0) {
            atomicOr(dev_status, NOVAKV_DEV_SMEM_LAYOUT);
            cta_range[blockIdx.x * 2] = 0; cta_range[blockIdx.x * 2 + 1] = 0;
        }
        return;
    }
    unsigned char* const t32_p = smem + C::OFFB_T32;
    unsigned char* const t16_p = smem + pad;
    unsigned char* const vcb_p = t16_p + (HAS16 ? T16_BYTES : 0);
    const uint32_t vcb_abs = t16_abs + (HAS16 ? T16_BYTES : 0);
    float* const q_s = reinterpret_cast<float*>(smem + C::OFFB_Q);
    const uint32_t s_p = s_base + C::OFFB_P;

    // With the KV-head-major walk the first KV head of CTA c is floor(c * Hkv / G) whatever the lengths are:
    // its (constant) value codebook starts flowing into shared memory before the grid-dependency wait and
    // lands behind the segment lookup and the first table build.
    int vcb_head = (int)(((long)blockIdx.x * n_kv_heads) / gridDim.x);   // KV head whose value codebook is resident
    stage_value_codebook_async<HAS16>(vcb_p, cb_v_img + (size_t)vcb_head * vcb_per_head);
    // With the merge fused in, the kernels that follow (the query transform of the next call writes the same
    // workspace) must not start before this grid is done: no early release of the dependents.
    if (out_fused != nullptr) asm volatile("griddepcontrol.wait;" ::: "memory");
    else novakv_grid_dependency_wait();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // The two prefixes are read many times (boundaries, segment look-ups): small batches keep them in shared memory.
    if (batch <= PFX_CAP) {
        int32_t* pfx = reinterpret_cast<int32_t*>(smem + C::OFFB_PFX);
        for (int i = threadIdx.x; i <= batch; i += S1_THREADS) { pfx[i] = page_prefix[i]; pfx[PFX_CAP + 1 + i] = cost_prefix[i]; }
        __syncthreads();
        page_prefix = pfx;
        cost_prefix = pfx + PFX_CAP + 1;
    }
    // First unit of every CTA (see scan_boundary): one thread per boundary.  This CTA owns [s_bnd[c], s_bnd[c + 1]).
    long* const s_bnd = reinterpret_cast<long*>(smem + C::OFFB_BND);
    for (int c = threadIdx.x; c <= (int)gridDim.x; c += S1_THREADS)
        s_bnd[c] = scan_boundary(c, gridDim.x, page_prefix, cost_prefix, batch, n_kv_heads, seg_weight);
    __syncthreads();
    const long u_begin = s_bnd[blockIdx.x], u_end = s_bnd[blockIdx.x + 1];
    if (threadIdx.x == 0) { cta_range[blockIdx.x * 2] = u_begin; cta_range[blockIdx.x * 2 + 1] = u_end; }
    if (u_begin >= u_end) { async_copies_wait(); return; }

    // ---- lane roles and constants
    const int fr = lane >> 2, fc = lane & 3;          // value side: MMA fragment coordinates
    // key side: token = lane; its byte j holds group j ^ (lane & 7) (j < 16) or j ^ (lane & 15) (j >= 16).
    //   binary32 entries (steps j < K32): address = T32 + code * ROW32 + ((j ^ lane%8) * 16): the column part is
    //     one xor with a constant away from a per-lane word, the row part one multiply-add;
    //   binary16 entries: address = T16 + code * 256 + ((j ^ mask) * 8) = a byte permutation of (index word,
    //     column word): the column word holds the column bytes of an even / odd step in bytes 0 / 1 and the
    //     table's upper address half in bytes 2, 3; stepping to another pair of j is one xor with a constant.
    const uint32_t col32 = s_base + C::OFFB_T32 + (lane & 7) * 16;
    const uint32_t colword15 = t16_abs | (uint32_t)((lane & 15) * 8) * 0x0101u;
    // value side: lane column fc reads copy fc / 2 of the value codebook; odd columns take the group blocks in
    // swapped order (x ^ 1), so that the 32 lanes of a gather hit 32 different slots.  With the binary16 table
    // (d = 128) the codebook block is 64 KB aligned too and its two copies share 256-byte rows, so that a gather
    // address is one byte permutation of (code word, pos); otherwise address = pos + code * 128.
    uint32_t pos[NGB];
#pragma unroll
    for (int x = 0; x < NGB; ++x) {
        const uint32_t slot4 = ((8 * (x ^ (fc & 1)) + fr + 16 * (fc >> 1)) & 31) * 4;
        pos[x] = HAS16 ? (vcb_abs | ((fc >> 1) * VCB_ROW + slot4)) : vcb_abs + (fc >> 1) * VCB_COPY_BYTES + slot4;
    }
    // address of the codeword whose code is byte b of word w, for load x
    auto vaddr = [&](uint32_t w, int b, int x) -> uint32_t {
        return HAS16 ? __byte_perm(w, pos[x], 0x7604u | (b << 4)) : pos[x] + __byte_perm(w, 0u, 0x4440u | b) * VCB_ROW;
    };
    const bool odd_col = fc & 1;
    // widening selectors: byte pairs (u, replicated top bit of u = 0) of the low / high half of a codeword, taken
    // from the first operand in even columns and from the second in odd columns
    const uint32_t sel_lo = odd_col ? 0xD5C4u : 0x9180u, sel_hi = odd_col ? 0xF7E6u : 0xB3A2u;
    // B fragments carry a weight in the low or high half depending on the column parity (fr & 1)
    const uint32_t sel_b0 = (fr & 1) ? 0x1044u : 0x4410u, sel_b1 = (fr & 1) ? 0x3244u : 0x4432u;
    const uint32_t s_pw = s_p + warp * C::P_WARP_BYTES;

    // ---- per-warp running state
    float m_run[HPAD];                           // running maximum of the logits (base 2), the same in every lane
    float macc[HSETS][NGB][4];                   //  VM: lane (fr, fc): head 4 hs + fc, group 8 gb + fr, 4 coefficients
    float wsum[HPAD];                            //  VM: this lane's tokens: sums of the (rounded) weights per head since the last offset removal
    float l_run[HPAD];                           //  VM: [hs] weight sum of head 4 hs + fc (every lane); else this lane's tokens, per head
    float lz_run[VSQ ? HPAD : 1];                //  VSQ: running sum_j p_j zero_j per head (this lane's tokens)
    uint64_t acc[VM ? 1 : NGB][VM ? 1 : HPAD][2];  // !VM: lane (fr, fc): group 8 gb + fr, head, 4 coefficients, its own tokens
    float esh_pow = 0.f;                         //  VSQ: 2^E with E >= log2 of every value scale seen so far (weights carry 2^-E)
#pragma unroll
    for (int h = 0; h < HPAD; ++h) { m_run[h] = M_INIT; l_run[h] = 0.f; }
#pragma unroll
    for (int h = 0; h < (VSQ ? HPAD : 1); ++h) lz_run[h] = 0.f;
#pragma unroll
    for (int hs = 0; hs < HSETS; ++hs) {
#pragma unroll
        for (int gb = 0; gb < NGB; ++gb)
#pragma unroll
            for (int i = 0; i < 4; ++i) macc[hs][gb][i] = 0.f;
    }
#pragma unroll
    for (int h = 0; h < HPAD; ++h) wsum[h] = 0.f;
#pragma unroll
    for (int x = 0; x < (VM ? 1 : NGB); ++x)
#pragma unroll
        for (int h = 0; h < (VM ? 1 : HPAD); ++h) { acc[x][h][0] = 0ull; acc[x][h][1] = 0ull; }

    // remove the centre of the value grid from the sums of the tiles since the last call (tensor-core value side)
    auto flush_window = [&]() {
        if (VSQ) return;          // INT2 levels carry no grid centre, and that format sums its normaliser per lane
#pragma unroll
        for (int hs = 0; hs < HSETS; ++hs) {
            // weight sum of head 4 hs + fc over the whole warp's tokens: transposing reduction inside the quad (each
            // step halves the heads a lane keeps), then a butterfly over the eight quads
            const float k0 = fc & 1 ? wsum[hs * 4 + 1] : wsum[hs * 4 + 0], s0 = fc & 1 ? wsum[hs * 4 + 0] : wsum[hs * 4 + 1];
            const float k1 = fc & 1 ? wsum[hs * 4 + 3] : wsum[hs * 4 + 2], s1 = fc & 1 ? wsum[hs * 4 + 2] : wsum[hs * 4 + 3];
            const float lo = k0 + __shfl_xor_sync(0xffffffffu, s0, 1), hi = k1 + __shfl_xor_sync(0xffffffffu, s1, 1);
            float w = (fc & 2 ? hi : lo) + __shfl_xor_sync(0xffffffffu, fc & 2 ? lo : hi, 2);
#pragma unroll
            for (int o = 4; o <= 16; o <<= 1) w += __shfl_xor_sync(0xffffffffu, w, o);
#pragma unroll
            for (int gb = 0; gb < NGB; ++gb)
#pragma unroll
                for (int i = 0; i < 4; ++i) macc[hs][gb][i] = fmaf(-CEN, w, macc[hs][gb][i]);
            l_run[hs] += w;
#pragma unroll
            for (int i = 0; i < 4; ++i) wsum[hs * 4 + i] = 0.f;
        }
    };

#ifdef NOVAKV_TIMING
    long long tm[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    unsigned long long g_start;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g_start));
    long long t_prev = clock64();
    const long long t_start = t_prev;
    int n_seg = 0;
#define NOVAKV_TICK(i) { const long long t_now = clock64(); tm[i] += t_now - t_prev; t_prev = t_now; }
#else
#define NOVAKV_TICK(i)
#endif
    long u = u_begin;
    while (u < u_end) {
        NOVAKV_TICK(0)
        const Segment sg = locate(page_prefix, seq_lens, batch, max_pages_per_seq, u, u_end, s_found);
        const int pair = sg.kvh * batch + sg.b;            // grows along the walk

        // ---- segment prologue -----------------------------------------------------------------
        if (vcb_head != sg.kvh) {
            stage_value_codebook_async<HAS16>(vcb_p, cb_v_img + (size_t)sg.kvh * vcb_per_head);
            vcb_head = sg.kvh;
        }
        // q' of the pair's heads -> shared memory (rows beyond HG are zero)
        for (int i = threadIdx.x; i < HPAD * D / 4; i += S1_THREADS) {
            const int h = i / (D / 4);
            const float4 v = h < HG ? reinterpret_cast<const float4*>(qp + ((size_t)sg.b * n_q_heads + sg.kvh * HG) * D)[i]
                                    : make_float4(0.f, 0.f, 0.f, 0.f);
            reinterpret_cast<float4*>(q_s)[i] = v;
        }
        float qcen[KSC ? HPAD : 1];
        if (KSC) {
#pragma unroll
            for (int h = 0; h < HPAD; ++h) qcen[h] = h < HG ? qc[(size_t)sg.b * n_q_heads + sg.kvh * HG + h] : 0.f;
        }

        // this warp's tiles of the segment: half pages hp = warp, warp + NCW, ...
        const int n_it = (2 * sg.npg > warp) ? (2 * sg.npg - warp + NCW - 1) / NCW : 0;
        const int32_t* pt = page_table + (size_t)sg.b * pt_stride + sg.pg0;
        // page ids of 32 consecutive tiles of this warp, one per lane (coalesced gather, loaded a batch ahead)
        auto load_ids = [&](int batch_i) {
            const int it = batch_i * 32 + lane;
            int page = 0;
            if (it < n_it) {
                page = pt[(warp + NCW * it) >> 1];
                if (page < 0 || page >= n_pages) { atomicOr(dev_status, NOVAKV_DEV_BAD_PAGE); page = 0; }
            }
            return page;
        };
        int ids_cur = load_ids(0), ids_next = load_ids(1);
        // tiles are loaded in ascending order, one ahead of the tile being consumed
        auto load_tile = [&](int it, TileRegs<L>& t) {
            if ((it & 31) == 0 && it > 0) { ids_cur = ids_next; ids_next = load_ids((it >> 5) + 1); }
            const int page = __shfl_sync(0xffffffffu, ids_cur, it & 31);
            const int half = (warp + NCW * it) & 1;
            const size_t off = ((size_t)page * n_kv_heads + sg.kvh) * PAGE_BYTES + half * TILE_BYTES;
            if (KSC) {
                const unsigned short raw = __ldg(reinterpret_cast<const unsigned short*>(k_scales) +
                                                 ((size_t)page * n_kv_heads + sg.kvh) * NOVAKV_PAGE_TOKENS + half * 32 + lane);
                t.ks = (uint32_t)raw << 16;
            }
            if (VSQ)
                t.vm = __ldg(reinterpret_cast<const uint32_t*>(v_meta) +
                             ((size_t)page * n_kv_heads + sg.kvh) * NOVAKV_PAGE_TOKENS + half * 32 + lane);
            const uint8_t* kp = k_pages + off + lane * 16;
            const uint8_t* vp = v_pages + off + lane * (NGB * 4);
#pragma unroll
            for (int p = 0; p < KPL; ++p) {
                const uint4 w = ldg_stream_128(kp + p * 512);
                t.kw[4 * p + 0] = w.x; t.kw[4 * p + 1] = w.y; t.kw[4 * p + 2] = w.z; t.kw[4 * p + 3] = w.w;
            }
#pragma unroll
            for (int blk = 0; blk < 2; ++blk) {
                if (NGB == 4) {
                    const uint4 w = ldg_stream_128(vp + blk * (L * 16));
                    t.vw[blk][0] = w.x; t.vw[blk][1] = w.y; t.vw[blk][NGB - 2] = w.z; t.vw[blk][NGB - 1] = w.w;
                } else {
                    const uint2 w = ldg_stream_64(vp + blk * (L * 16));
                    t.vw[blk][0] = w.x; t.vw[blk][1] = w.y;
                }
            }
        };

        // ---- one 32-token tile -------------------------------------------------------------------
        auto process = [&](const TileRegs<L>& cur, int it) {
            const int hp = warp + NCW * it;
            const int tok0 = (sg.pg0 + (hp >> 1)) * NOVAKV_PAGE_TOKENS + (hp & 1) * 32;
            const int nvalid = min(32, sg.len - tok0);
            if (nvalid <= 0) return;

            // ---- key side: lane <-> token; step j gathers the entry of (code_j, group j ^ lane bits) ------
            float zf[HPAD];
            {
                uint64_t z2[HPAD / 2];
#pragma unroll
                for (int k = 0; k < HPAD / 2; ++k) z2[k] = 0ull;
#pragma unroll
                for (int j = 0; j < K32; ++j) {
                    const uint32_t code = __byte_perm(cur.kw[j >> 2], 0u, 0x4440u | (j & 3));
                    const uint32_t a = (col32 ^ (uint32_t)(j * 16)) + code * C::ROW32;
#pragma unroll
                    for (int hs = 0; hs < HSETS; ++hs) {
                        const uint4 v = lds_u128(a + hs * C::PLANE32);
                        fadd2(z2[2 * hs], (uint64_t)v.x | ((uint64_t)v.y << 32));
                        fadd2(z2[2 * hs + 1], (uint64_t)v.z | ((uint64_t)v.w << 32));
                    }
                }
#pragma unroll
                for (int k = 0; k < HPAD / 2; ++k) unpack2(z2[k], zf[2 * k], zf[2 * k + 1]);
            }
            if (HAS16) {
                // (with a per-token key scale the sum is multiplied by rho afterwards, which carries the rounding of the
                // binary16 chains into tokens of large norm: shorter chains there)
                constexpr int CHAIN = KSC ? NOVAKV_KSC_CHAIN : NOVAKV_CHAIN;
                uint32_t ch[2];
#pragma unroll
                for (int j = K32; j < L; ++j) {
                    const uint32_t cw2 = colword15 ^ (uint32_t)(((j & ~1) * 8) | (((j | 1) * 8) << 8));
                    const uint2 v = lds_u64(__byte_perm(cur.kw[j >> 2], cw2, 0x7600u | ((j & 3) << 4) | (4 + (j & 1))));
                    if ((j - K32) % CHAIN == 0) { ch[0] = v.x; ch[1] = v.y; }
                    else { ch[0] = hadd2(ch[0], v.x); ch[1] = hadd2(ch[1], v.y); }
                    if ((j - K32) % CHAIN == CHAIN - 1 || j == L - 1) {
                        flush_h2(ch[0], zf[0], zf[1]);
                        flush_h2(ch[1], zf[2], zf[3]);
                    }
                }
            }
            float vscale = 1.f, vzero = 0.f, vsmax = 0.f;     // vsmax: this lane's scale as it enters the running bound (0 beyond the length)
            if (KSC) {
                const float rho = __uint_as_float(cur.ks);
#pragma unroll
                for (int h = 0; h < HPAD; ++h) zf[h] = (zf[h] + qcen[h]) * rho;
            }
            if (VSQ && lane < nvalid) {
                // (slots beyond the length hold no metadata; a scale that is not positive and finite counts as 1)
                vscale = __uint_as_float(cur.vm << 16);
                vzero = __uint_as_float(cur.vm & 0xffff0000u);
                if (!(vscale > 0.f && vscale < CUDART_INF_F)) vscale = 1.f;
                vsmax = vscale;
            }
            if (nvalid < 32 && lane >= nvalid) {
#pragma unroll
                for (int h = 0; h < HPAD; ++h) zf[h] = -CUDART_INF_F;
            }
            // ---- online softmax (base 2): the running maximum moves only when a logit exceeds it ---------
            {
                bool up = false;
#pragma unroll
                for (int h = 0; h < HPAD; ++h) up |= zf[h] > m_run[h];
                if (VSQ) up |= vsmax >= esh_pow;
                if (__any_sync(0xffffffffu, up)) {
                    float alpha[HPAD];
#pragma unroll
                    for (int h = 0; h < HPAD; ++h) {
                        // a head whose maximum moved gets M_SLACK bits of headroom above the new maximum: the next
                        // few record logits then need no update (the reference point of a softmax is free; weights
                        // stay <= 2^SH, and those below 2^(SH - 24 + M_SLACK) of the maximum vanish)
                        const float wm = warp_max(zf[h]);
                        const float m_new = wm > m_run[h] ? wm + M_SLACK : m_run[h];
                        alpha[h] = ex2(m_run[h] - m_new);
                        m_run[h] = m_new;
                    }
                    float vsc = 1.f;                     // VSQ: 2^(E_old - E_new)
                    if (VSQ) {
                        // E = exponent of the largest scale so far + 1 (scale < 2^E), an exact power of two
                        const float smax = warp_max(vsmax);
                        const float e_new = __uint_as_float((__float_as_uint(smax) & 0x7f800000u) + 0x00800000u);
                        if (e_new > esh_pow) { vsc = esh_pow / e_new; esh_pow = e_new; }
                    }
                    if (VM) {
#pragma unroll
                        for (int hs = 0; hs < HSETS; ++hs) {
                            const float a01 = fc & 1 ? alpha[hs * 4 + 1] : alpha[hs * 4 + 0];
                            const float a23 = fc & 1 ? alpha[hs * 4 + 3] : alpha[hs * 4 + 2];
                            const float al = fc & 2 ? a23 : a01;
#pragma unroll
                            for (int gb = 0; gb < NGB; ++gb)
#pragma unroll
                                for (int i = 0; i < 4; ++i) macc[hs][gb][i] *= al * vsc;
                            if (!VSQ) {
                                l_run[hs] *= al;
                                // the weight sums still waiting for their window flush move with the accumulators
#pragma unroll
                                for (int i = 0; i < 4; ++i) wsum[hs * 4 + i] *= alpha[hs * 4 + i];
                            }
                        }
                        if (VSQ) {
#pragma unroll
                            for (int h = 0; h < HPAD; ++h) { l_run[h] *= alpha[h]; lz_run[h] *= alpha[h]; }
                        }
                    } else {
#pragma unroll
                        for (int h = 0; h < HPAD; ++h) {
                            const uint64_t a2 = pack2(alpha[h], alpha[h]);
#pragma unroll
                            for (int x = 0; x < NGB; ++x) { fmul2(acc[VM ? 0 : x][VM ? 0 : h][0], a2); fmul2(acc[VM ? 0 : x][VM ? 0 : h][1], a2); }
                            l_run[h] *= alpha[h];
                        }
                    }
                }
            }
            // weights
            uint32_t ph[HPAD / 2];
            if (VSQ) {
                // INT2 values: the tensor-core product needs the weight of the token's integer codes,
                // w = p * scale (times 2^15 / 2^E), in binary16.  The rounding must not separate numerator and
                // normaliser: the weight that counts is p' = fp16(w) / (scale 2^-E), used for the normaliser and
                // for the zero-point sum as well (an exact softmax of perturbed logits).
                const float wmul = __fdividef(vscale, esh_pow), winv = __fdividef(esh_pow, vscale);
#pragma unroll
                for (int h = 0; h < HPAD; h += 2) {
                    const float w0 = ex2(zf[h] - m_run[h] + SH) * wmul, w1 = ex2(zf[h + 1] - m_run[h + 1] + SH) * wmul;
                    ph[h / 2] = pack_h2(w0, w1);
                    const float2 wf = __half22float2(*reinterpret_cast<const __half2*>(&ph[h / 2]));
                    const float p0 = wf.x * winv, p1 = wf.y * winv;
                    l_run[h] += p0; l_run[h + 1] += p1;
                    lz_run[h] = fmaf(p0, vzero, lz_run[h]); lz_run[h + 1] = fmaf(p1, vzero, lz_run[h + 1]);
                }
            } else if (VM) {
#pragma unroll
                for (int h = 0; h < HPAD; h += 2)
                {
                    ph[h / 2] = pack_h2(ex2(zf[h] - m_run[h] + SH), ex2(zf[h + 1] - m_run[h + 1] + SH));
                    flush_h2(ph[h / 2], wsum[h], wsum[h + 1]);       // the rounded weights are what the normaliser sums
                }
            } else {
#pragma unroll
                for (int h = 0; h < HPAD; ++h) { zf[h] = ex2(zf[h] - m_run[h]); l_run[h] += zf[h]; }
            }

            if (VM) {
                // ---- value side on tensor cores ---------------------------------------------------------
                // D[m][n] += sum_k A[m][k] B[k][n], m16 n8 k16, per 8-token sub-tile and group block gb:
                //   k = (token j of the sub-tile, sub-coefficient i in {0,1}),
                //   A[m][(j,i)] = 2^-24 x grid index of codeword(token j, group 8gb + (m & 7))[2 (m >> 3) + i]     fp16 (subnormal)
                //   B[(j,i)][(h,i')] = w_h(token j) * [i == i']                                                fp16
                //   D[m][(h,i')] = partial of head h, group 8gb + (m & 7), coefficient 2 (m >> 3) + i'
                // weights -> shared memory as fp16, [head][k-slot pair = token & 3][token >> 3, (token >> 2) & 1]
                __syncwarp();      // previous tile's readers of the P area are done
                {
                    const uint32_t wa = s_pw + (lane & 3) * 16 + ((lane >> 3) * 2 + ((lane >> 2) & 1)) * 2;
#pragma unroll
                    for (int h = 0; h < HPAD; ++h)
                        asm volatile("st.shared.u16 [%0], %1;" ::"r"(wa + h * 64),
                                     "h"((unsigned short)((h & 1) ? (ph[h / 2] >> 16) : (ph[h / 2] & 0xffffu))) : "memory");
                }
                __syncwarp();
                // B-fragment sources: 8 weights of head (4 hs + fr/2) for the tokens with (token & 3) == fc
                uint4 pw[HSETS];
#pragma unroll
                for (int hs = 0; hs < HSETS; ++hs) pw[hs] = lds_u128(s_pw + (hs * 4 + (fr >> 1)) * 64 + fc * 16);
#pragma unroll
                for (int blk = 0; blk < 2; ++blk) {
#pragma unroll
                    for (int ts = 0; ts < 2; ++ts) {                       // 8-token sub-tiles of the block
                        const int t = blk * 2 + ts;                         // sub-tile index within the 32-token tile
                        uint32_t b0[HSETS], b1[HSETS];
#pragma unroll
                        for (int hs = 0; hs < HSETS; ++hs) {
                            const uint32_t w = t == 0 ? pw[hs].x : (t == 1 ? pw[hs].y : (t == 2 ? pw[hs].z : pw[hs].w));
                            b0[hs] = __byte_perm(w, 0u, sel_b0);
                            b1[hs] = __byte_perm(w, 0u, sel_b1);
                        }
                        // gather: X[x][u] = codeword of token 8ts + 4u + fc of the block, group block x ^ (fc & 1), row fr
                        uint32_t X[NGB][2];
#pragma unroll
                        for (int x = 0; x < NGB; ++x) {
                            const uint32_t vwd = cur.vw[blk][x];      // codes of the group block this load fetches (x ^ 1 in odd columns)
                            X[x][0] = lds_u32(vaddr(vwd, 2 * ts, x));
                            X[x][1] = lds_u32(vaddr(vwd, 2 * ts + 1, x));
                        }
#pragma unroll
                        for (int gb = 0; gb < NGB; ++gb) {
                            // bytes (u, 0) pairs from X[gb] (even columns) or X[gb ^ 1] (odd columns)
                            const uint32_t a0 = prmt_rep(X[gb][0], X[gb ^ 1][0], sel_lo), a1 = prmt_rep(X[gb][0], X[gb ^ 1][0], sel_hi);
                            const uint32_t a2 = prmt_rep(X[gb][1], X[gb ^ 1][1], sel_lo), a3 = prmt_rep(X[gb][1], X[gb ^ 1][1], sel_hi);
#pragma unroll
                            for (int hs = 0; hs < HSETS; ++hs) mma_f16(macc[hs][gb], a0, a1, a2, a3, b0[hs], b1[hs]);
                        }
                    }
                }
                if ((it & (NOVAKV_WINDOW - 1)) == NOVAKV_WINDOW - 1) flush_window();
            } else {
                // ---- value side on CUDA cores (fp32): same lane coordinates and gathers, FMA instead of MMA ----
                __syncwarp();      // previous tile's readers of the P area are done
#pragma unroll
                for (int h = 0; h < HPAD; h += 4)
                    asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(s_pw + lane * (HPAD * 4) + h * 4),
                                 "f"(zf[h]), "f"(zf[h + 1]), "f"(zf[h + 2]), "f"(zf[h + 3]) : "memory");
                __syncwarp();
#pragma unroll
                for (int blk = 0; blk < 2; ++blk)
#pragma unroll
                    for (int tq = 0; tq < 4; ++tq) {                       // this lane's 4 tokens of the block: 4 tq + fc
                        const int tok = blk * 16 + tq * 4 + fc;
                        float pf[HPAD];
#pragma unroll
                        for (int h = 0; h < HPAD; h += 4)
                            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(pf[h]), "=f"(pf[h + 1]), "=f"(pf[h + 2]), "=f"(pf[h + 3])
                                         : "r"(s_pw + tok * (HPAD * 4) + h * 4));
#pragma unroll
                        for (int x = 0; x < NGB; ++x) {
                            // (odd lane columns fetch group block x ^ 1 with load x; their accumulator x holds that block)
                            const uint32_t cwd = lds_u32(vaddr(cur.vw[blk][x], tq, x));
                            // grid indices -> binary32, centred: bytes (u, 0) are the binary16 subnormals u 2^-24
                            const __half2 c64 = __halves2half2(__ushort_as_half((unsigned short)64), __ushort_as_half((unsigned short)64));
                            const uint32_t h01 = __byte_perm(cwd, 0u, 0x4140u), h23 = __byte_perm(cwd, 0u, 0x4342u);
                            const float2 f01 = __half22float2(__hsub2(*reinterpret_cast<const __half2*>(&h01), c64));
                            const float2 f23 = __half22float2(__hsub2(*reinterpret_cast<const __half2*>(&h23), c64));
                            const uint64_t v01 = pack2(f01.x, f01.y), v23 = pack2(f23.x, f23.y);
#pragma unroll
                            for (int h = 0; h < HPAD; ++h) {
                                const uint64_t p2 = pack2(pf[h], pf[h]);
                                ffma2(acc[VM ? 0 : x][VM ? 0 : h][0], v01, p2);
                                ffma2(acc[VM ? 0 : x][VM ? 0 : h][1], v23, p2);
                            }
                        }
                    }
            }
        };

        // ---- score table (the first tile's loads are issued before, so that they fly during the build)
        TileRegs<L> ta;
        if (n_it > 0) load_tile(0, ta);
        __syncthreads();     // q' of the pair is in shared memory
        NOVAKV_TICK(1)
        build_score_table<D, HG, VM>(t32_p, t16_p, cb_k_lut + (size_t)sg.kvh * 256 * L * 4, q_s);
        NOVAKV_TICK(2)
        async_copies_wait();
        __syncthreads();     // table and value codebook complete
        NOVAKV_TICK(3)

        // ---- scan: 32-token tiles, the next tile's loads in flight while one is consumed
        for (int it = 0; it < n_it; ++it) {
            const TileRegs<L> cur = ta;
            if (it + 1 < n_it) load_tile(it + 1, ta);
            process(cur, it);
        }

        // ---- segment epilogue: merge the warps' partials, write one partial ---------------------
        NOVAKV_TICK(4)
        if (VM) flush_window();
        __syncthreads();                                   // scan done everywhere: the tables are dead
        NOVAKV_TICK(5)
        unsigned char* const merge_p = HAS16 ? t16_p : t32_p;
        float* m_acc = reinterpret_cast<float*>(merge_p);                              // [NCW][HPAD][MROW]
        float* m_ml = reinterpret_cast<float*>(merge_p + C::MERGE_ACC_BYTES);          // [NCW][HPAD][2]
        float* m_lz = m_ml + NCW * HPAD * 2;                                           // [NCW][HPAD]  (VSQ)
        if (VM && !VSQ) {
            // lane (fr = 0, fc) holds the weight sum of heads 4 hs + fc
            if (fr == 0) {
#pragma unroll
                for (int hs = 0; hs < HSETS; ++hs) {
                    const float ma01 = fc & 1 ? m_run[hs * 4 + 1] : m_run[hs * 4 + 0];
                    const float ma23 = fc & 1 ? m_run[hs * 4 + 3] : m_run[hs * 4 + 2];
                    m_ml[(warp * HPAD + hs * 4 + fc) * 2] = fc & 2 ? ma23 : ma01;
                    m_ml[(warp * HPAD + hs * 4 + fc) * 2 + 1] = l_run[hs];
                }
            }
        } else {
#pragma unroll
            for (int h = 0; h < HPAD; ++h) {
                const float lsum = warp_sum(l_run[h]);
                if (lane == 0) { m_ml[(warp * HPAD + h) * 2] = m_run[h]; m_ml[(warp * HPAD + h) * 2 + 1] = lsum; }
                if (VSQ) {
                    const float lz = warp_sum(lz_run[h]);
                    if (lane == 0) m_lz[warp * HPAD + h] = lz;
                    lz_run[h] = 0.f;
                }
            }
        }
#pragma unroll
        for (int h = 0; h < HPAD; ++h) { m_run[h] = M_INIT; l_run[h] = 0.f; }
        if (VM) {
            // VSQ: the sums carry 2^-E of the scales; E is per warp, so it is folded back here
            const float unsh = VSQ ? esh_pow : 1.f;
#pragma unroll
            for (int hs = 0; hs < HSETS; ++hs)
#pragma unroll
                for (int gb = 0; gb < NGB; ++gb) {
                    *reinterpret_cast<float4*>(m_acc + ((size_t)warp * HPAD + hs * 4 + fc) * C::MROW + (8 * gb + fr) * 4) =
                        make_float4(macc[hs][gb][0] * unsh, macc[hs][gb][1] * unsh, macc[hs][gb][2] * unsh, macc[hs][gb][3] * unsh);
#pragma unroll
                    for (int i = 0; i < 4; ++i) macc[hs][gb][i] = 0.f;
                }
            esh_pow = 0.f;
        } else {
            // every lane column holds a partial over its own tokens (accumulator x of an odd column belongs to group
            // block x ^ 1): add the four columns, column fc writes head 4 k + fc
#pragma unroll
            for (int x = 0; x < NGB; ++x) {
#pragma unroll
                for (int h = 0; h < HPAD; ++h) {
                    float a0, a1, a2, a3, b0, b1, b2, b3;
                    unpack2(acc[VM ? 0 : x][VM ? 0 : h][0], a0, a1);
                    unpack2(acc[VM ? 0 : x][VM ? 0 : h][1], a2, a3);
                    unpack2(acc[VM ? 0 : (x ^ 1)][VM ? 0 : h][0], b0, b1);
                    unpack2(acc[VM ? 0 : (x ^ 1)][VM ? 0 : h][1], b2, b3);
                    if (odd_col) { a0 = b0; a1 = b1; a2 = b2; a3 = b3; }           // now: this lane's partial of group block x
#pragma unroll
                    for (int o = 1; o <= 2; o <<= 1) {
                        a0 += __shfl_xor_sync(0xffffffffu, a0, o); a1 += __shfl_xor_sync(0xffffffffu, a1, o);
                        a2 += __shfl_xor_sync(0xffffffffu, a2, o); a3 += __shfl_xor_sync(0xffffffffu, a3, o);
                    }
                    if ((h & 3) == fc)
                        *reinterpret_cast<float4*>(m_acc + ((size_t)warp * HPAD + h) * C::MROW + (8 * x + fr) * 4) = make_float4(a0, a1, a2, a3);
                }
            }
#pragma unroll
            for (int x = 0; x < NGB; ++x)
#pragma unroll
                for (int h = 0; h < HPAD; ++h) { acc[VM ? 0 : x][VM ? 0 : h][0] = 0ull; acc[VM ? 0 : x][VM ? 0 : h][1] = 0ull; }
        }
        __syncthreads();
        {
            const size_t pidx = (size_t)pair + blockIdx.x;      // unique: pair and CTA index both grow along the walk
            const float unscale = VM ? 3.0517578125e-05f : 1.f;  // 2^-15: the weights carried 2^15
            for (int i = threadIdx.x; i < HG * D; i += S1_THREADS) {
                const int h = i / D, c = i - h * D;
                float M = M_INIT;
#pragma unroll
                for (int w = 0; w < NCW; ++w) M = fmaxf(M, m_ml[(w * HPAD + h) * 2]);
                float a = 0.f, lsum = 0.f, zsum = 0.f;
#pragma unroll
                for (int w = 0; w < NCW; ++w) {
                    const float sc = ex2(m_ml[(w * HPAD + h) * 2] - M);
                    a = fmaf(sc, m_acc[((size_t)w * HPAD + h) * C::MROW + c], a);
                    if (VSQ) zsum = fmaf(sc, m_lz[w * HPAD + h], zsum);              // zero-points: the same amount on every coefficient
                    lsum = fmaf(sc, m_ml[(w * HPAD + h) * 2 + 1], lsum);
                }
                // grid index sums -> value-transform coefficients: s (u - 64) + (lo + 64 s) per unit of weight
                a *= 16777216.f;                           // indices entered the sums as u 2^-24
                float val;
                if (VSQ) val = (a + zsum) * unscale;       // levels are the codes themselves (s = 1, no offset)
                else val = (v_scale[(size_t)sg.kvh * D + c] * a + v_off[(size_t)sg.kvh * D + c] * lsum) * unscale;
                part_acc[(pidx * HG + h) * D + c] = val;
                if (c == 0) { part_ml[(pidx * HG + h) * 2] = M; part_ml[(pidx * HG + h) * 2 + 1] = lsum * unscale; }
            }
        }
        if (out_fused != nullptr) {
            // arrival: this CTA's partial is visible before its count is; the CTA that completes the count merges
            __threadfence();
            __syncthreads();
            if (threadIdx.x == 0) {
                s_arrived = atomicAdd(&pair_count[pair], 1) + 1;
                s_first = gridDim.x;
                s_last = -1;
            }
            __syncthreads();
            const long P = page_prefix[batch];
            const long pu0 = (long)sg.kvh * P + page_prefix[sg.b], pu1 = pu0 + (sg.len + NOVAKV_PAGE_TOKENS - 1) / NOVAKV_PAGE_TOKENS;
            bool touches = false;                           // CTA threadIdx.x has a non-empty share of this pair
            if (threadIdx.x < gridDim.x) {
                const int c = threadIdx.x;
                touches = s_bnd[c] < s_bnd[c + 1] && s_bnd[c] < pu1 && s_bnd[c + 1] > pu0;
                if (touches) { atomicMin(&s_first, c); atomicMax(&s_last, c); }
            }
            const int expected = __syncthreads_count(touches);
            if (s_arrived == expected) {
                __threadfence();
                fused_merge<D, HG>(reinterpret_cast<float*>(t32_p), part_ml, part_acc, pair, s_first, s_last, s_bnd, rv_t, v_mean,
                                   sg.kvh, out_fused, out_is_fp32, ((size_t)sg.b * n_q_heads + sg.kvh * HG) * D);
                if (threadIdx.x == 0) pair_count[pair] = 0;
            }
        }
        __syncthreads();                                   // merge buffer free before the next table build
        NOVAKV_TICK(6)
#ifdef NOVAKV_TIMING
        ++n_seg;
#endif
        u += sg.npg;
    }
#ifdef NOVAKV_TIMING
    unsigned long long g_end;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g_end));
    if (threadIdx.x == 0)
        printf("cta %3d segs %d pages %ld | clocks: pre-loop %lld locate+q %lld build %lld vcbwait %lld scan(w0) %lld barrier %lld epilogue %lld total %lld | ns start %llu end %llu\n",
               blockIdx.x, n_seg, (long)(u_end - u_begin), tm[0], tm[1], tm[2], tm[3], tm[4], tm[5], tm[6], clock64() - t_start, g_start, g_end);
#endif
}

// ------------------------------------------------------------------------------------------------
// merge + inverse value transform
// ------------------------------------------------------------------------------------------------
// MINB = resident blocks per SM the register budget allows for: 1 keeps the prefetched constants in
// registers (lowest latency, small batches), 2 trades a few spills for occupancy (many pairs).
// EXT = the call carries a learned sink logit and/or a BF16 band partial; without it that code is compiled out.
template <int D, int HG, int MINB, bool EXT>
__global__ void __launch_bounds__(HG * D > 512 ? 512 : HG * D, MINB)
novakv_decode_merge_kernel(const float* __restrict__ part_ml, const float* __restrict__ part_acc,
                           const int32_t* __restrict__ page_prefix, const int32_t* __restrict__ seq_lens,
                           int batch, int n_q_heads, int n_kv_heads, int max_pages_per_seq, int grid_s1,
                           const float* __restrict__ rv_t, const float* __restrict__ v_mean,
                           void* __restrict__ out, int out_is_fp32,
                           const float* __restrict__ sink_logits /* [Hq] natural-log units, or null */,
                           const float* __restrict__ qk_off /* [batch][Hq], base-2 units */,
                           const float* __restrict__ band_ml /* [batch][Hq][2] (max, sum) of the BF16 band, or null */,
                           const float* __restrict__ band_acc /* [batch][Hq][D] sum p v of the band, original value domain */,
                           const int32_t* __restrict__ cost_prefix, int seg_weight, const long* __restrict__ cta_range) {
    __shared__ float o_s[HG * D];
    __shared__ float frac_s[HG];      // share of the softmax mass on quantised tokens (1 without sink and band)
    __shared__ float bsc_s[HG];       // multiplier of the band accumulator (0 without a band)
    constexpr int NT = HG * D > 512 ? 512 : HG * D;
    constexpr int PARTS = NT / D, COLS = D / PARTS;
    const int pair = blockIdx.x;
    const int b = pair / n_kv_heads, kvh = pair - b * n_kv_heads;
    // constants of the inverse transform are fetched before the grid-dependency wait (they overlap the
    // tail of the scan kernel): this thread's slice of rv_t and the mean of its output coordinates
    float rv[COLS];
    {
        const float* R = rv_t + (size_t)kvh * D * D + (size_t)(threadIdx.x / D) * COLS * D + threadIdx.x % D;   // rv_t[c][r] = R_V[r][c]
#pragma unroll
        for (int c = 0; c < COLS; ++c) rv[c] = R[(size_t)c * D];
    }
    float vm[(HG * D + NT - 1) / NT];
#pragma unroll
    for (int k = 0; k < (HG * D + NT - 1) / NT; ++k) vm[k] = v_mean[(size_t)kvh * D + (threadIdx.x + k * NT) % D];
#ifdef NOVAKV_TIMING
    unsigned long long g_m0, g_m1, g_m2;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g_m0));
#endif
    novakv_grid_dependency_wait();
#ifdef NOVAKV_TIMING
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g_m1));
#endif
    const int len = clamp_len(seq_lens[b], max_pages_per_seq);
    const int pages_b = (len + NOVAKV_PAGE_TOKENS - 1) / NOVAKV_PAGE_TOKENS;
    const long P = page_prefix[batch];
    const int slot0 = kvh * batch + b;                     // the scan kernel's pair index (walk order)
    // CTAs that may hold a piece of this pair: those whose cost range meets the pair's (the largest c with
    // floor(c*T/G) <= x for its first and last cost unit), widened by one on each side; the ranges the scan
    // CTAs recorded decide.  Their ranges, then their (max, sum) pairs, are fetched into shared memory by
    // parallel threads (two memory latencies, whatever the number of pieces), so that the loop below only issues
    // independent loads of the accumulators.
    __shared__ int cand_s[MAX_SCAN_CTAS + 1];              // 1 = this CTA holds a piece of the pair
    __shared__ float2 ml_s[MAX_SCAN_CTAS + 1][HG];
    int c_first = 0, n_cand = 0;
    if (pages_b > 0) {
        const long u0 = (long)kvh * P + page_prefix[b], u1 = u0 + pages_b;
        const long T = (long)cost_prefix[batch] * n_kv_heads;
        const long x0 = (long)kvh * cost_prefix[batch] + cost_prefix[b] + seg_weight, x1 = x0 + pages_b - 1;
        c_first = max((int)(((x0 + 1) * grid_s1 - 1) / T) - 1, 0);
        const int c_last = min((int)(((x1 + 1) * grid_s1 - 1) / T) + 1, grid_s1 - 1);
        n_cand = min(c_last - c_first + 1, MAX_SCAN_CTAS + 1);
        for (int t = threadIdx.x; t < n_cand; t += blockDim.x) {
            const long r0 = cta_range[(c_first + t) * 2], r1 = cta_range[(c_first + t) * 2 + 1];
            cand_s[t] = (r0 < r1 && r1 > u0 && r0 < u1) ? 1 : 0;
        }
        __syncthreads();
        for (int t = threadIdx.x; t < n_cand * HG; t += blockDim.x) {
            const int ci = t / HG, h = t - ci * HG;
            if (cand_s[ci]) ml_s[ci][h] = *reinterpret_cast<const float2*>(part_ml + (((size_t)slot0 + c_first + ci) * HG + h) * 2);
        }
        __syncthreads();
    }
    for (int i = threadIdx.x; i < HG * D; i += blockDim.x) {
        const int h = i / D, c = i - h * D;
        float M = M_INIT, a = 0.f, lsum = 0.f;
        for (int ci = 0; ci < n_cand; ++ci)
            if (cand_s[ci]) M = fmaxf(M, ml_s[ci][h].x);
        for (int ci = 0; ci < n_cand; ++ci) {
            if (!cand_s[ci]) continue;
            const float sc = ex2(ml_s[ci][h].x - M);
            a = fmaf(sc, part_acc[(((size_t)slot0 + c_first + ci) * HG + h) * D + c], a);
            lsum = fmaf(sc, ml_s[ci][h].y, lsum);
        }
        float lq = lsum;          // mass of the quantised tokens at the running scale
        float wb = 0.f;           // weight of the band accumulator at the running scale
        const int hq = kvh * HG + h;
        if (EXT && band_ml != nullptr) {
            // BF16 sink-plus-recent band: one more partial, accumulated in the original value domain
            const float mb = band_ml[((size_t)b * n_q_heads + hq) * 2], lb = band_ml[((size_t)b * n_q_heads + hq) * 2 + 1];
            const float M2 = fmaxf(M, mb);
            const float wq = ex2(M - M2);
            wb = ex2(mb - M2);
            a *= wq;
            lq *= wq;
            lsum = fmaf(lb, wb, lq);
            M = M2;
        }
        if (EXT && sink_logits != nullptr) {
            // learned sink: an extra logit in the normaliser, added exactly once, after the cross-split
            // combine; it is shifted by the per-query constant the token logits dropped (q . k_mean)
            const float s2 = sink_logits[hq] * 1.4426950408889634f - qk_off[(size_t)b * n_q_heads + hq];
            const float M2 = fmaxf(M, s2);
            const float w = ex2(M - M2);
            a *= w;
            lq *= w;
            wb *= w;
            lsum = fmaf(lsum, w, ex2(s2 - M2));
        }
        float val = 0.f, frac = 0.f, bsc = 0.f;
        if (lsum > 0.f) {
            val = a / lsum;
            if (EXT) { frac = lq / lsum; bsc = wb / lsum; }
        }
        if (EXT && c == 0) { frac_s[h] = frac; bsc_s[h] = bsc; }
        o_s[i] = val;
    }
    __syncthreads();
    // o_h = o'_h rv^T + v_mean: threads = D outputs x PARTS column parts, all HG heads share each load
    __shared__ float red_s[PARTS][HG][D];
    {
        const int r = threadIdx.x % D, part = threadIdx.x / D;
        float acc[HG];
#pragma unroll
        for (int h = 0; h < HG; ++h) acc[h] = 0.f;
        if (pages_b > 0) {
#pragma unroll
            for (int c = 0; c < COLS; ++c)
#pragma unroll
                for (int h = 0; h < HG; ++h) acc[h] = fmaf(o_s[h * D + part * COLS + c], rv[c], acc[h]);
        }
#pragma unroll
        for (int h = 0; h < HG; ++h) red_s[part][h][r] = acc[h];
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < (HG * D + NT - 1) / NT; ++k) {
        const int i = threadIdx.x + k * NT;
        if (i >= HG * D) break;
        const int h = i / D, r = i - h * D;
        float o = 0.f;
#pragma unroll
        for (int p = 0; p < PARTS; ++p) o += red_s[p][h][r];
        // sum_j p_j (s^_j R_V^T + v_mean): the mean carries the quantised-token mass (all of it without sink and band)
        if (EXT) o = fmaf(vm[k], frac_s[h], o);
        else if (pages_b > 0) o += vm[k];
        const size_t oi = ((size_t)b * n_q_heads + kvh * HG + h) * D + r;
        if (EXT && band_acc != nullptr) o = fmaf(band_acc[oi], bsc_s[h], o);
        if (out_is_fp32) reinterpret_cast<float*>(out)[oi] = o;
        else reinterpret_cast<__nv_bfloat16*>(out)[oi] = __float2bfloat16_rn(o);
    }
#ifdef NOVAKV_TIMING
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g_m2));
    if (threadIdx.x == 0 && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1))
        printf("merge block %d | ns start %llu after-wait %llu end %llu\n", blockIdx.x, g_m0, g_m1, g_m2);
#endif
}

// ------------------------------------------------------------------------------------------------
// BF16 sink-plus-recent band: exact attention partial over the tokens that are not quantised
// ------------------------------------------------------------------------------------------------
// One CTA per (sequence, KV head), 16 warps; a warp takes 4 band tokens at a time (their 8 row loads in
// flight together), lanes hold D/32 dimensions, logits by warp reduction, online softmax per warp, then a
// merge of the warps.  Output: (max, sum) and sum_j p_j v_j per query head, base-2 domain, unnormalised.
// Band buffers: bf16 [batch][band_cap][Hkv][D]; of sequence b, slots 0 .. sink_cnt-1 hold the sink tokens
// and slots n_sink + (ring_start + i) % (band_cap - n_sink), i < ring_len, the recent tokens.
constexpr int BAND_WARPS = 16, BAND_U = 4;
template <int D, int HG>
__global__ void __launch_bounds__(BAND_WARPS * 32)
novakv_band_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ band_k,
                   const __nv_bfloat16* __restrict__ band_v, int band_cap, int n_sink,
                   const int32_t* __restrict__ band_meta, int n_q_heads, int n_kv_heads, float scale_log2,
                   const float* __restrict__ k_mean, float* __restrict__ band_ml, float* __restrict__ band_acc) {
    constexpr int DPL = D / 32;
    __shared__ float m_s[BAND_WARPS][HG], l_s[BAND_WARPS][HG];
    __shared__ float acc_s[BAND_WARPS][HG][D];
    novakv_grid_dependency_wait();
    const int b = blockIdx.x / n_kv_heads, kvh = blockIdx.x - b * n_kv_heads;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ring_cap = band_cap - n_sink;
    const int sink_cnt = min(max(band_meta[b * 3 + 0], 0), n_sink);
    const int ring_start = max(band_meta[b * 3 + 1], 0);
    const int ring_len = ring_cap > 0 ? min(max(band_meta[b * 3 + 2], 0), ring_cap) : 0;
    const int n = sink_cnt + ring_len;
    float qr[HG][DPL];
#pragma unroll
    for (int h = 0; h < HG; ++h)
#pragma unroll
        for (int i = 0; i < DPL; ++i)
            qr[h][i] = __bfloat162float(q[((size_t)b * n_q_heads + kvh * HG + h) * D + lane * DPL + i]) * scale_log2;
    // the quantised tokens' logits omit the constant q . k_mean * sm_scale (Lemma S1): the band's logits must
    // sit on the same scale, so the same constant is subtracted here
    float zoff[HG];
#pragma unroll
    for (int h = 0; h < HG; ++h) {
        float t = 0.f;
#pragma unroll
        for (int i = 0; i < DPL; ++i) t = fmaf(qr[h][i], k_mean[(size_t)kvh * D + lane * DPL + i], t);
        zoff[h] = warp_sum_f(t);
    }
    float m[HG], l[HG], acc[HG][DPL];
#pragma unroll
    for (int h = 0; h < HG; ++h) {
        m[h] = M_INIT; l[h] = 0.f;
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[h][i] = 0.f;
    }
    for (int base = warp * BAND_U; base < n; base += BAND_WARPS * BAND_U) {
        float kf[BAND_U][DPL], vf[BAND_U][DPL];
#pragma unroll
        for (int u = 0; u < BAND_U; ++u) {
            const int i = base + u;
            const int ii = i < n ? i : base;               // a valid row; its weight is zeroed below
            const int slot = ii < sink_cnt ? ii : n_sink + (ring_start + (ii - sink_cnt)) % ring_cap;
            const size_t off = (((size_t)b * band_cap + slot) * n_kv_heads + kvh) * D + lane * DPL;
#pragma unroll
            for (int j = 0; j < DPL; j += 2) {
                const __nv_bfloat162 k2 = *reinterpret_cast<const __nv_bfloat162*>(band_k + off + j);
                const __nv_bfloat162 v2 = *reinterpret_cast<const __nv_bfloat162*>(band_v + off + j);
                kf[u][j] = __bfloat162float(k2.x); kf[u][j + 1] = __bfloat162float(k2.y);
                vf[u][j] = __bfloat162float(v2.x); vf[u][j + 1] = __bfloat162float(v2.y);
            }
        }
#pragma unroll
        for (int u = 0; u < BAND_U; ++u) {
            const bool valid = base + u < n;
#pragma unroll
            for (int h = 0; h < HG; ++h) {
                float z = 0.f;
#pragma unroll
                for (int i = 0; i < DPL; ++i) z = fmaf(qr[h][i], kf[u][i], z);
                z = warp_sum_f(z) - zoff[h];
                if (!valid) z = -CUDART_INF_F;
                const float m_new = fmaxf(m[h], z);
                const float alpha = ex2(m[h] - m_new), p = ex2(z - m_new);
                l[h] = fmaf(l[h], alpha, p);
#pragma unroll
                for (int i = 0; i < DPL; ++i) acc[h][i] = fmaf(acc[h][i], alpha, p * vf[u][i]);
                m[h] = m_new;
            }
        }
    }
#pragma unroll
    for (int h = 0; h < HG; ++h) {
        if (lane == 0) { m_s[warp][h] = m[h]; l_s[warp][h] = l[h]; }
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc_s[warp][h][lane * DPL + i] = acc[h][i];
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < HG * D; idx += BAND_WARPS * 32) {
        const int h = idx / D, c = idx - h * D;
        float M = M_INIT;
#pragma unroll
        for (int w = 0; w < BAND_WARPS; ++w) M = fmaxf(M, m_s[w][h]);
        float a = 0.f, L = 0.f;
#pragma unroll
        for (int w = 0; w < BAND_WARPS; ++w) {
            const float sc = ex2(m_s[w][h] - M);
            a = fmaf(sc, acc_s[w][h][c], a);
            L = fmaf(sc, l_s[w][h], L);
        }
        const size_t o = (size_t)b * n_q_heads + kvh * HG + h;
        band_acc[o * D + c] = a;
        if (c == 0) { band_ml[o * 2] = M; band_ml[o * 2 + 1] = L; }
    }
}

// workspace layout
struct WsLayout {
    size_t qp, prefix, cost, range, qk, qc, cnt, bml, bacc, ml, acc, total;
};
WsLayout ws_layout(const novakv_ctx* ctx, int batch) {
    auto al = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t d = ctx->cfg.head_dim, hq = ctx->cfg.n_q_heads;
    const size_t n_part = (size_t)batch * ctx->cfg.n_kv_heads + ctx->n_sm;
    WsLayout w;
    w.qp = 0;
    w.prefix = al(w.qp + (size_t)batch * hq * d * 4);
    w.cost = al(w.prefix + ((size_t)batch + 1) * 4);
    w.range = al(w.cost + ((size_t)batch + 1) * 4);
    w.qk = al(w.range + (size_t)ctx->n_sm * 2 * sizeof(long));
    w.qc = al(w.qk + (size_t)batch * hq * 4);
    w.cnt = al(w.qc + (size_t)batch * hq * 4);
    w.bml = al(w.cnt + (size_t)batch * ctx->cfg.n_kv_heads * 4);
    w.bacc = al(w.bml + (size_t)batch * hq * 2 * 4);
    w.ml = al(w.bacc + (size_t)batch * hq * d * 4);
    w.acc = al(w.ml + n_part * ctx->hg * 2 * 4);
    w.total = al(w.acc + n_part * ctx->hg * d * 4);
    return w;
}

template <int D, int HG, bool VM, bool KSC, bool VSQ>
novakv_status launch_decode_t(novakv_ctx* ctx, const novakv_layer& ly, const __nv_bfloat16* q,
                              const uint8_t* k_pages, const uint8_t* v_pages, const __nv_bfloat16* k_scales,
                              const __nv_bfloat16* v_meta, int n_pages,
                              const int32_t* page_table, int max_pages_per_seq, const int32_t* seq_lens,
                              int batch, float sm_scale, void* out, int out_is_fp32, void* workspace,
                              cudaStream_t stream, const float* sink_logits, const novakv_band_args* band) {
    using C = S1<D, HG, VM>;
    // with a BF16 band the index cache holds positions n_sink .. n_sink + seq_lens[b] - 1: the scan starts at
    // page column n_sink / 64 of every row
    const int pt_stride = max_pages_per_seq;
    if (band != nullptr) {
        const int shift = band->n_sink / NOVAKV_PAGE_TOKENS;
        page_table += shift;
        max_pages_per_seq -= shift;
    }
    const WsLayout w = ws_layout(ctx, batch);
    char* ws = (char*)workspace;
    float* qp = (float*)(ws + w.qp);
    int32_t* prefix = (int32_t*)(ws + w.prefix);
    int32_t* cost_prefix = (int32_t*)(ws + w.cost);
    long* cta_range = (long*)(ws + w.range);
    float* qk_off = sink_logits ? (float*)(ws + w.qk) : nullptr;
    float* qc = KSC ? (float*)(ws + w.qc) : nullptr;
    // what the token logits drop: q . k_mean, and for the unscaled key format also the share of the codebook
    // centres (k_mean_eff = k_mean + centre R_K^{-1}); with a per-token scale the centres are added back instead
    const float* k_off_vec = KSC ? ly.k_mean : ly.k_mean_eff;
    float* band_ml = band ? (float*)(ws + w.bml) : nullptr;
    float* band_acc = band ? (float*)(ws + w.bacc) : nullptr;
    float* part_ml = (float*)(ws + w.ml);
    float* part_acc = (float*)(ws + w.acc);
    int32_t* pair_count = (int32_t*)(ws + w.cnt);
    const int hq = ctx->cfg.n_q_heads, hkv = ctx->cfg.n_kv_heads;
    const int grid = ctx->scan_ctas > 0 ? (ctx->scan_ctas < ctx->n_sm ? ctx->scan_ctas : ctx->n_sm) : ctx->n_sm;
    if (grid > MAX_SCAN_CTAS) return NOVAKV_EUNSUPPORTED;
    // Optionally (novakv_debug_set_fused_merge), without a sink logit or a BF16 band, the scan kernel merges each
    // (sequence, KV head) pair itself (the CTA that writes the pair's last partial does it); otherwise the merge
    // kernel follows.
    const bool fuse = sink_logits == nullptr && band == nullptr && ctx->fused_merge;

    novakv_launch_pdl(novakv_prepare_kernel<D, HG>, dim3(batch * hkv + 1), dim3(512), 0, stream, q, ly.rk_inv_t, seq_lens,
                      batch, hq, hkv, max_pages_per_seq, sm_scale * 1.4426950408889634f, qp, prefix, ctx->dev_status,
                      k_off_vec, qk_off, cost_prefix, ctx->seg_weight, (const float*)ly.k_center, qc,
                      fuse ? pair_count : (int32_t*)nullptr, fuse ? out : (void*)nullptr, out_is_fp32);
    ctx->launches++;

    auto kern = novakv_decode_stage1_kernel<D, HG, VM, KSC, VSQ>;
    // the opt-in is per device and per kernel instantiation: remembered in the context (one device each)
    constexpr unsigned inst_bit = 1u << ((VM ? 1 : 0) + (KSC ? 2 : 0) + (VSQ ? 4 : 0));
    if (!(ctx->smem_opt_in & inst_bit)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, S1_SMEM_BYTES) != cudaSuccess) return NOVAKV_ECUDA;
        ctx->smem_opt_in |= inst_bit;
    }
    {
        novakv_prof_scope ps(ctx, 0, stream);
        novakv_launch_pdl(kern, dim3(grid), dim3(S1_THREADS), S1_SMEM_BYTES, stream, qp, ly.cb_k_lut,
                          VSQ ? (const uint8_t*)ctx->int2_img : (const uint8_t*)ly.cb_v_u8, (const float*)ly.v_scale,
                          (const float*)ly.v_off, k_pages, v_pages, k_scales, v_meta, n_pages, page_table, max_pages_per_seq,
                          seq_lens, prefix, batch, hq, hkv, part_ml, part_acc, ctx->dev_status, pt_stride,
                          (const int32_t*)cost_prefix, ctx->seg_weight, cta_range, (const float*)qc,
                          VSQ ? 0 : VCB_COPY_BYTES, pair_count, (const float*)ly.rv_t, (const float*)ly.v_mean,
                          fuse ? out : (void*)nullptr, out_is_fp32);
        ps.end();
        ctx->launches++;
    }
    if (band != nullptr) {
        novakv_launch_pdl(novakv_band_kernel<D, HG>, dim3(batch * hkv), dim3(BAND_WARPS * 32), 0, stream, q, band->k, band->v,
                          band->cap, band->n_sink, band->meta, hq, hkv, sm_scale * 1.4426950408889634f, k_off_vec, band_ml,
                          band_acc);
        ctx->launches++;
    }
    if (fuse) return cudaGetLastError() == cudaSuccess ? NOVAKV_OK : NOVAKV_ECUDA;
    const bool ext = sink_logits != nullptr || band != nullptr;
    auto merge = batch * hkv > 2 * ctx->n_sm
                     ? (ext ? novakv_decode_merge_kernel<D, HG, 2, true> : novakv_decode_merge_kernel<D, HG, 2, false>)
                     : (ext ? novakv_decode_merge_kernel<D, HG, 1, true> : novakv_decode_merge_kernel<D, HG, 1, false>);
    novakv_launch_pdl(merge, dim3(batch * hkv), dim3(HG * D > 512 ? 512 : HG * D), 0, stream,
                      part_ml, part_acc, prefix, seq_lens, batch, hq, hkv, max_pages_per_seq, grid, ly.rv_t, ly.v_mean, out,
                      out_is_fp32, sink_logits, qk_off, (const float*)band_ml, (const float*)band_acc,
                      (const int32_t*)cost_prefix, ctx->seg_weight, (const long*)cta_range);
    ctx->launches++;
    return cudaGetLastError() == cudaSuccess ? NOVAKV_OK : NOVAKV_ECUDA;
}

}  // namespace

size_t novakv_decode_ws_bytes(const novakv_ctx* ctx, int batch) { return ws_layout(ctx, batch).total; }

novakv_status novakv_launch_decode(novakv_ctx* ctx, const novakv_layer& ly, const __nv_bfloat16* q,
    const uint8_t* k_pages, const uint8_t* v_pages, int n_pages, const int32_t* page_table,
    int max_pages_per_seq, const int32_t* seq_lens, int batch, float sm_scale, void* out,
    int out_is_fp32, void* workspace, size_t workspace_bytes, cudaStream_t stream, const __nv_bfloat16* k_scales,
    const float* sink_logits, const novakv_band_args* band, const __nv_bfloat16* v_meta) {
    (void)workspace_bytes;
    const int d = ctx->cfg.head_dim, hg = ctx->hg;
    if (k_scales != nullptr && ctx->value_path == 0) return NOVAKV_EUNSUPPORTED;   // scaled keys: tensor-core value side only
    if (v_meta != nullptr && k_scales == nullptr) return NOVAKV_EUNSUPPORTED;      // INT2 values come with scaled keys (deployed format)
#define NOVAKV_DISPATCH(DD, HH)                                                                             \
    if (d == DD && hg == HH) {                                                                                   \
        if (v_meta != nullptr)                                                                                   \
            return launch_decode_t<DD, HH, true, true, true>(ctx, ly, q, k_pages, v_pages, k_scales, v_meta, n_pages, page_table, \
                                                  max_pages_per_seq, seq_lens, batch, sm_scale, out, out_is_fp32, \
                                                  workspace, stream, sink_logits, band);                         \
        if (k_scales != nullptr)                                                                                 \
            return launch_decode_t<DD, HH, true, true, false>(ctx, ly, q, k_pages, v_pages, k_scales, nullptr, n_pages, page_table, \
                                                  max_pages_per_seq, seq_lens, batch, sm_scale, out, out_is_fp32, \
                                                  workspace, stream, sink_logits, band);                               \
        if (ctx->value_path == 0)                                                                                \
            return launch_decode_t<DD, HH, false, false, false>(ctx, ly, q, k_pages, v_pages, nullptr, nullptr, n_pages, page_table, \
                                                  max_pages_per_seq, seq_lens, batch, sm_scale, out, out_is_fp32, \
                                                  workspace, stream, sink_logits, band);                               \
        return launch_decode_t<DD, HH, true, false, false>(ctx, ly, q, k_pages, v_pages, nullptr, nullptr, n_pages, page_table,  \
                                             max_pages_per_seq, seq_lens, batch, sm_scale, out, out_is_fp32,     \
                                             workspace, stream, sink_logits, band);                                    \
    }
    NOVAKV_DISPATCH(128, 1)
    NOVAKV_DISPATCH(128, 2)
    NOVAKV_DISPATCH(128, 4)
    NOVAKV_DISPATCH(64, 1)
    NOVAKV_DISPATCH(64, 2)
    NOVAKV_DISPATCH(64, 4)
    NOVAKV_DISPATCH(64, 8)
#undef NOVAKV_DISPATCH
    return NOVAKV_ESHAPE;
}
