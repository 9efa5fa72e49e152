// Internal declarations shared by the translation units of libnovakv (not installed).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <vector>

#include "novakv.h"

#define NOVAKV_PAGE_TOKENS 64
#define NOVAKV_G 4
#define NOVAKV_C 256
#define NOVAKV_VBLOCK 16

// Device copies of one layer's tables, in the layouts the kernels read.
struct novakv_layer {
    bool loaded = false;
    // write path (binary64 transforms, see the encode entry of the public header)
    double* rk_d = nullptr;       // [Hkv][d][d]
    double* rv_d = nullptr;       // [Hkv][d][d]
    double* rk_d_mma = nullptr;   // [Hkv][d/4][d][4]: rk_d with the input dimension blocked by 4 (tensor-core fragments)
    double* rv_d_mma = nullptr;   // same for rv_d
    double* k_mean_d = nullptr;   // [Hkv][d]
    float* k_mean = nullptr;      // [Hkv][d] (offset q . k_mean of a sink logit / the BF16 band, scaled key format)
    float* k_mean_eff = nullptr;  // [Hkv][d] k_mean + centre R_K^{-1}: the same offset when the table is built from centred codewords
    float* k_center = nullptr;    // [Hkv][d] per (group, coordinate) midrange of the key codewords (transform domain)
    double* v_mean_d = nullptr;   // [Hkv][d]
    float* cb_k = nullptr;        // [Hkv][L][256][4]  search layout
    float* cb_v = nullptr;        // [Hkv][L][256][4]
    // read path
    float* rk_inv_t = nullptr;    // [Hkv][d][d]
    float* rv_t = nullptr;        // [Hkv][d][d]  transposed R_V: rv_t[c][r] = R_V[r][c]
    float* v_mean = nullptr;      // [Hkv][d]
    float* cb_k_lut = nullptr;    // [Hkv][256][L][4]   key codewords minus k_center, the order the score table is built in
    uint8_t* cb_v_u8 = nullptr;   // [Hkv][256][32][4]  value codewords as indices (0..127) of their 7-bit grid, slot = group
    float* v_scale = nullptr;     // [Hkv][d]  grid step s of each value coefficient: codeword = lo + s u
    float* v_off = nullptr;       // [Hkv][d]  lo + 128 s
};

struct novakv_event_pair {
    cudaEvent_t start, stop;
};

struct novakv_ctx {
    novakv_config cfg;
    int hg = 0, n_groups = 0, n_sm = 0;
    std::vector<novakv_layer> layers;
    uint32_t* dev_status = nullptr;
    void* int2_img = nullptr;     // uint8 [256][32][4]: the product codebook {0,1,2,3}^4 in the value-gather layout
    bool profile = false;
    std::vector<novakv_event_pair> prof[3];
    std::vector<novakv_event_pair> prof_free;
    long launches = 0;
    int scan_ctas = 0;            // 0 = one per SM
    int value_path = 1;           // 1 = tensor cores, 0 = CUDA cores
    int seg_weight = 24;          // pages one (sequence, KV head) segment weighs extra in the scan kernel's work split
    bool fused_merge = false;     // true: the scan kernel merges the partials itself where it can (no sink, no band)
    unsigned smem_opt_in = 0;     // scan-kernel instantiations whose shared-memory opt-in was set on this device
};

// RAII-free helper: brackets a launch with events when profiling is on.
struct novakv_prof_scope {
    novakv_ctx* ctx;
    int kind;
    cudaStream_t stream;
    novakv_event_pair ev;
    bool active;
    novakv_prof_scope(novakv_ctx* c, int k, cudaStream_t s);
    void end();
};

// encode
novakv_status novakv_launch_encode(novakv_ctx* ctx, const novakv_layer& ly, const __nv_bfloat16* k_new,
    const __nv_bfloat16* v_new, const int32_t* tok_seq, const int32_t* tok_pos, int n_tokens,
    uint8_t* k_pages, uint8_t* v_pages, int n_pages, const int32_t* page_table,
    int max_pages_per_seq, int n_seq, int32_t* seq_lens, cudaStream_t stream,
    __nv_bfloat16* k_scales = nullptr /* scaled key format: [n_pages][Hkv][64] */,
    __nv_bfloat16* v_meta = nullptr /* INT2 value codec: (scale, zero) [n_pages][Hkv][64][2] */);
novakv_status novakv_launch_search(novakv_ctx* ctx, const novakv_layer& ly, int which, const float* coef,
    int n, uint8_t* idx_out, cudaStream_t stream);

// decode
struct novakv_band_args {
    const __nv_bfloat16* k;     // [batch][cap][Hkv][d]
    const __nv_bfloat16* v;
    int cap;                    // slots per sequence: n_sink sink slots + a ring of cap - n_sink
    int n_sink;                 // multiple of 64
    const int32_t* meta;        // device [batch][3]: sink count, ring start, ring length
};
size_t novakv_decode_ws_bytes(const novakv_ctx* ctx, int batch);
novakv_status novakv_launch_decode(novakv_ctx* ctx, const novakv_layer& ly, const __nv_bfloat16* q,
    const uint8_t* k_pages, const uint8_t* v_pages, int n_pages, const int32_t* page_table,
    int max_pages_per_seq, const int32_t* seq_lens, int batch, float sm_scale, void* out,
    int out_is_fp32, void* workspace, size_t workspace_bytes, cudaStream_t stream,
    const __nv_bfloat16* k_scales = nullptr /* scaled key format: [n_pages][Hkv][64] */,
    const float* sink_logits = nullptr /* learned sink: [Hq], natural-log units */,
    const novakv_band_args* band = nullptr /* BF16 sink-plus-recent band */,
    const __nv_bfloat16* v_meta = nullptr /* INT2 value codec: (scale, zero) [n_pages][Hkv][64][2] */);

// gather of page-locked host buffers into device staging (one kernel for up to 5 segments of 32-bit words)
struct novakv_stage_args {
    const uint32_t* src[5];
    uint32_t* dst[5];
    unsigned words[5];
    int n;
};
novakv_status novakv_launch_stage(novakv_ctx* ctx, const novakv_stage_args& a, cudaStream_t stream);
novakv_status novakv_launch_band_insert(novakv_ctx* ctx, const void* k_new, const void* v_new, int batch, void* band_k,
    void* band_v, int band_cap, int n_sink, int n_rec, int block, int32_t* band_meta, int32_t* quant_lens,
    void* stage_k, void* stage_v, int32_t* tok_seq, int32_t* tok_pos, cudaStream_t stream);

// bf16 comparator
size_t novakv_bf16_ws_bytes(const novakv_ctx* ctx, int batch, int max_pages_per_seq);
novakv_status novakv_launch_bf16_decode(novakv_ctx* ctx, const __nv_bfloat16* q,
    const __nv_bfloat16* k_pages, const __nv_bfloat16* v_pages, int n_pages,
    const int32_t* page_table, int max_pages_per_seq, const int32_t* seq_lens, int batch,
    float sm_scale, int window, void* out, int out_is_fp32, void* workspace, size_t workspace_bytes,
    cudaStream_t stream);

// ---------------------------------------------------------------- device helpers
#ifdef __CUDACC__

// Programmatic dependent launch: a kernel launched with novakv_launch_pdl may be scheduled while its
// predecessor in the stream is still running; it must call novakv_grid_dependency_wait() before it
// touches anything a preceding kernel may write, which blocks until the predecessor grid has completed
// and its writes are visible.  Before the wait a kernel only reads calibration constants (uploaded
// synchronously by novakv_load_calibration, never written by a kernel) into registers or its own shared
// memory, so the launch latency and that staging overlap the predecessor's tail.  There is no unbounded
// wait in user code.
__device__ __forceinline__ void novakv_grid_dependency_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename... KArgs, typename... Args>
cudaError_t novakv_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Byte offsets inside the 64*L-byte chunk of one (page, KV head); t = token slot in the page
// (0..63), l = group.  These define the cache format (see the public header).
//   keys:   [tile = t/32][plane][token t%32][16 bytes]; byte j of a token's L bytes (plane j/16) holds
//           the code of group j ^ (t % 8) for j < 16 and of group j ^ (t % 16) for j >= 16.
//   values: [block = t/16][fr = l%8][fc = t%4][gb = l/8][b = (t%16)/4].
template <int L>
__host__ __device__ __forceinline__ int novakv_k_offset(int t, int l) {
    constexpr int KPL = L / 16;
    const int j = l ^ (t & (l < 16 ? 7 : 15));
    return (((t >> 5) * KPL + (j >> 4)) * 32 + (t & 31)) * 16 + (j & 15);
}
template <int L>
__host__ __device__ __forceinline__ int novakv_v_offset(int t, int l) {
    constexpr int NGB = L / 8;
    const int tb = t & 15, fc = tb & 3, b = tb >> 2, fr = l & 7;
    return (t >> 4) * (L * 16) + (fr * 4 + fc) * (NGB * 4) + ((l >> 3) ^ (fc & 1)) * 4 + b;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

#endif  // __CUDACC__
