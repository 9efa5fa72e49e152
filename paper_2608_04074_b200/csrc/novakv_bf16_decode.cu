// Uncompressed comparator: the same decode step on a bf16 paged cache (textbook attention, Eq.
// "scores"), used only to report the compression speed-up on identical shapes and to serve the
// sliding-window layers of hybrid models, which the paper leaves in bf16 (Sec. 5).
//
// Split over the sequence like the quantised path: grid (split, KV head, sequence), each CTA scans
// BF16_SPLIT_PAGES pages; a merge kernel combines the splits.  HBM-bound by design (512 bytes per
// token and KV head at d = 128): every lane owns d/32 dimensions of the head, keys and values are read
// with coalesced loads (one token row per warp instruction), the logits of 8 tokens x Hg heads are
// reduced across lanes with one transposed butterfly (31 shuffles instead of 160).
#include <math_constants.h>

#include "novakv_internal.cuh"

namespace {

constexpr int BF16_SPLIT_PAGES = 16;     // 1024 tokens per CTA
constexpr int BF16_WARPS = 4;
constexpr int TG = 8;                    // tokens per warp iteration
constexpr float M_INIT = -1.0e30f;

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int N>
__device__ __forceinline__ void butterfly_step(float (&v)[N], int s, int lane) {
    // lanes with bit s set keep the upper half, the others the lower half; the kept half receives the
    // partner's contribution to it
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
        const bool up = (lane & s) != 0;
        const float send = up ? v[i] : v[i + N / 2];
        const float keep = up ? v[i + N / 2] : v[i];
        v[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
    }
}

// DPL = dims per lane (4 at d = 128, 2 at d = 64)
template <int DPL>
struct RowChunk {
    uint32_t w[DPL / 2];
};
template <int DPL>
__device__ __forceinline__ RowChunk<DPL> load_chunk(const __nv_bfloat16* p) {
    RowChunk<DPL> r;
    if (DPL == 4) {
        const uint2 v = *reinterpret_cast<const uint2*>(p);
        r.w[0] = v.x; r.w[DPL / 2 - 1] = v.y;
    } else {
        r.w[0] = *reinterpret_cast<const uint32_t*>(p);
    }
    return r;
}
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

template <int D, int HG>
__global__ void __launch_bounds__(BF16_WARPS * 32)
novakv_bf16_stage1_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k_pages,
                          const __nv_bfloat16* __restrict__ v_pages, int n_pages,
                          const int32_t* __restrict__ page_table, int max_pages_per_seq,
                          const int32_t* __restrict__ seq_lens, int n_q_heads, int n_kv_heads, float scale_log2,
                          int window, int max_splits, float* __restrict__ part_ml, float* __restrict__ part_acc) {
    constexpr int DPL = D / 32;
    constexpr int NV = TG * HG;              // logits per warp iteration
    constexpr int VPL = NV / 32;             // of which each lane finishes VPL (1 at Hg = 4, 2 at Hg = 8)
    static_assert(NV % 32 == 0, "Hg must be 4 or 8");
    const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int len = seq_lens[b];
    len = len < 0 ? 0 : min(len, max_pages_per_seq * NOVAKV_PAGE_TOKENS);
    const int start = window > 0 ? max(0, len - window) : 0;
    const int first_page = start / NOVAKV_PAGE_TOKENS;
    const int t_begin = (first_page + split * BF16_SPLIT_PAGES) * NOVAKV_PAGE_TOKENS;
    const int t_end = min(len, t_begin + BF16_SPLIT_PAGES * NOVAKV_PAGE_TOKENS);
    if (t_begin >= t_end) return;

    // q of the Hg heads, this lane's dims, pre-scaled into the base-2 domain
    float qr[HG][DPL];
#pragma unroll
    for (int h = 0; h < HG; ++h)
#pragma unroll
        for (int i = 0; i < DPL; ++i)
            qr[h][i] = __bfloat162float(q[((size_t)b * n_q_heads + kvh * HG + h) * D + lane * DPL + i]) * scale_log2;

    float acc[HG][DPL];
#pragma unroll
    for (int h = 0; h < HG; ++h)
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[h][i] = 0.f;
    // this lane finishes the logits with flat index lane*VPL + j = token*HG + head
    float m_run[VPL], l_run[VPL];
#pragma unroll
    for (int j = 0; j < VPL; ++j) { m_run[j] = M_INIT; l_run[j] = 0.f; }

    const int n_groups = (t_end - t_begin + TG - 1) / TG;
    auto row_ptr = [&](const __nv_bfloat16* pool, int tok) {
        int page = page_table[(size_t)b * max_pages_per_seq + tok / NOVAKV_PAGE_TOKENS];
        page = (page < 0 || page >= n_pages) ? 0 : page;
        return pool + (((size_t)page * n_kv_heads + kvh) * NOVAKV_PAGE_TOKENS + tok % NOVAKV_PAGE_TOKENS) * D + lane * DPL;
    };
    RowChunk<DPL> kn[TG], vn[TG];
    auto load_group = [&](int g) {
        const int tok0 = t_begin + g * TG;             // 8-token groups never straddle a page
        const __nv_bfloat16* kp = row_ptr(k_pages, tok0);
        const __nv_bfloat16* vp = row_ptr(v_pages, tok0);
#pragma unroll
        for (int t = 0; t < TG; ++t) { kn[t] = load_chunk<DPL>(kp + (size_t)t * D); vn[t] = load_chunk<DPL>(vp + (size_t)t * D); }
    };
    if (warp < n_groups) load_group(warp);
    for (int g = warp; g < n_groups; g += BF16_WARPS) {
        RowChunk<DPL> kc[TG], vc[TG];
#pragma unroll
        for (int t = 0; t < TG; ++t) { kc[t] = kn[t]; vc[t] = vn[t]; }
        if (g + BF16_WARPS < n_groups) load_group(g + BF16_WARPS);
        const int tok0 = t_begin + g * TG;
        // partial dot products of this lane's dims: z[token*HG + head]
        float z[NV];
#pragma unroll
        for (int t = 0; t < TG; ++t)
#pragma unroll
            for (int h = 0; h < HG; ++h) {
                float s = qr[h][0] * bf16lo(kc[t].w[0]);
                s = fmaf(qr[h][1], bf16hi(kc[t].w[0]), s);
                if (DPL == 4) {
                    s = fmaf(qr[h][DPL - 2], bf16lo(kc[t].w[DPL / 2 - 1]), s);
                    s = fmaf(qr[h][DPL - 1], bf16hi(kc[t].w[DPL / 2 - 1]), s);
                }
                z[t * HG + h] = s;
            }
        // transposed butterfly: afterwards lane holds the complete logits lane*VPL + j
        {
            float (&v32)[NV] = z;
            butterfly_step<NV>(v32, 16, lane);
            float (&v16)[NV / 2] = reinterpret_cast<float (&)[NV / 2]>(z);
            butterfly_step<NV / 2>(v16, 8, lane);
            float (&v8)[NV / 4] = reinterpret_cast<float (&)[NV / 4]>(z);
            butterfly_step<NV / 4>(v8, 4, lane);
            float (&v4)[NV / 8] = reinterpret_cast<float (&)[NV / 8]>(z);
            butterfly_step<NV / 8>(v4, 2, lane);
            float (&v2)[NV / 16] = reinterpret_cast<float (&)[NV / 16]>(z);
            butterfly_step<NV / 16>(v2, 1, lane);
        }
        // online softmax; the lanes that share a head differ in the lane bits above log2(HG / VPL)
        float p[VPL], alpha[VPL];
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            const int flat = lane * VPL + j, t = flat / HG;
            float zz = z[j];
            if (tok0 + t >= t_end || tok0 + t < start) zz = -CUDART_INF_F;
            float mx = zz;
#pragma unroll
            for (int s = HG / VPL; s < 32; s <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
            const float m_new = fmaxf(m_run[j], mx);
            alpha[j] = ex2f(m_run[j] - m_new);
            m_run[j] = m_new;
            p[j] = ex2f(zz - m_new);
            l_run[j] = fmaf(l_run[j], alpha[j], p[j]);
        }
        // rescale and accumulate values: every lane needs alpha and p of all heads and tokens
#pragma unroll
        for (int h = 0; h < HG; ++h) {
            const float a = __shfl_sync(0xffffffffu, alpha[h % VPL], h / VPL);     // head h lives at flat index h (token 0)
#pragma unroll
            for (int i = 0; i < DPL; ++i) acc[h][i] *= a;
        }
#pragma unroll
        for (int t = 0; t < TG; ++t) {
            float vv[DPL];
            vv[0] = bf16lo(vc[t].w[0]); vv[1] = bf16hi(vc[t].w[0]);
            if (DPL == 4) { vv[DPL - 2] = bf16lo(vc[t].w[DPL / 2 - 1]); vv[DPL - 1] = bf16hi(vc[t].w[DPL / 2 - 1]); }
            if (tok0 + t >= t_end || tok0 + t < start) {      // bytes past the sequence are arbitrary: keep 0 * NaN out
#pragma unroll
                for (int i = 0; i < DPL; ++i) vv[i] = 0.f;
            }
#pragma unroll
            for (int h = 0; h < HG; ++h) {
                const int flat = t * HG + h;
                const float ph = __shfl_sync(0xffffffffu, p[flat % VPL], flat / VPL);
#pragma unroll
                for (int i = 0; i < DPL; ++i) acc[h][i] = fmaf(ph, vv[i], acc[h][i]);
            }
        }
    }

    // ---- merge the 4 warps and write the split's partial ---------------------------------------
    __shared__ float s_acc[BF16_WARPS][HG][D];
    __shared__ float s_ml[BF16_WARPS][HG][2];
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
        float l = l_run[j];
#pragma unroll
        for (int s = HG / VPL; s < 32; s <<= 1) l += __shfl_xor_sync(0xffffffffu, l, s);
        const int flat = lane * VPL + j;
        if (flat < HG) { s_ml[warp][flat][0] = m_run[j]; s_ml[warp][flat][1] = l; }
    }
#pragma unroll
    for (int h = 0; h < HG; ++h)
#pragma unroll
        for (int i = 0; i < DPL; ++i) s_acc[warp][h][lane * DPL + i] = acc[h][i];
    __syncthreads();
    const size_t pidx = ((size_t)(b * n_kv_heads + kvh) * max_splits + split);
    for (int i = threadIdx.x; i < HG * D; i += BF16_WARPS * 32) {
        const int h = i / D, c = i % D;
        float M = M_INIT;
#pragma unroll
        for (int w = 0; w < BF16_WARPS; ++w) M = fmaxf(M, s_ml[w][h][0]);
        float a = 0.f, l = 0.f;
#pragma unroll
        for (int w = 0; w < BF16_WARPS; ++w) {
            const float sc = ex2f(s_ml[w][h][0] - M);
            a = fmaf(sc, s_acc[w][h][c], a);
            l = fmaf(sc, s_ml[w][h][1], l);
        }
        part_acc[(pidx * HG + h) * D + c] = a;
        if (c == 0) { part_ml[(pidx * HG + h) * 2] = M; part_ml[(pidx * HG + h) * 2 + 1] = l; }
    }
}

template <int D, int HG>
__global__ void novakv_bf16_merge_kernel(const float* __restrict__ part_ml, const float* __restrict__ part_acc,
                                         const int32_t* __restrict__ seq_lens, int max_pages_per_seq, int n_q_heads,
                                         int n_kv_heads, int window, int max_splits, void* __restrict__ out,
                                         int out_is_fp32) {
    const int pair = blockIdx.x, b = pair / n_kv_heads, kvh = pair % n_kv_heads;
    int len = seq_lens[b];
    len = len < 0 ? 0 : min(len, max_pages_per_seq * NOVAKV_PAGE_TOKENS);
    const int start = window > 0 ? max(0, len - window) : 0;
    const int first_page = start / NOVAKV_PAGE_TOKENS;
    const int pages = (len + NOVAKV_PAGE_TOKENS - 1) / NOVAKV_PAGE_TOKENS - first_page;
    const int n_splits = len > 0 ? (pages + BF16_SPLIT_PAGES - 1) / BF16_SPLIT_PAGES : 0;
    for (int i = threadIdx.x; i < HG * D; i += blockDim.x) {
        const int h = i / D, c = i % D;
        float o = 0.f;
        if (n_splits > 0) {
            float M = M_INIT;
            for (int s = 0; s < n_splits; ++s) M = fmaxf(M, part_ml[((((size_t)pair * max_splits + s) * HG + h)) * 2]);
            float a = 0.f, l = 0.f;
            for (int s = 0; s < n_splits; ++s) {
                const size_t pidx = (size_t)pair * max_splits + s;
                const float sc = ex2f(part_ml[(pidx * HG + h) * 2] - M);
                a = fmaf(sc, part_acc[(pidx * HG + h) * D + c], a);
                l = fmaf(sc, part_ml[(pidx * HG + h) * 2 + 1], l);
            }
            o = a / l;
        }
        const size_t oi = ((size_t)b * n_q_heads + kvh * HG + h) * D + c;
        if (out_is_fp32) reinterpret_cast<float*>(out)[oi] = o;
        else reinterpret_cast<__nv_bfloat16*>(out)[oi] = __float2bfloat16_rn(o);
    }
}

int max_splits_of(int max_pages_per_seq) { return (max_pages_per_seq + BF16_SPLIT_PAGES - 1) / BF16_SPLIT_PAGES + 1; }

template <int D, int HG>
novakv_status launch_bf16_t(novakv_ctx* ctx, const __nv_bfloat16* q, const __nv_bfloat16* k_pages,
                            const __nv_bfloat16* v_pages, int n_pages, const int32_t* page_table,
                            int max_pages_per_seq, const int32_t* seq_lens, int batch, float sm_scale, int window,
                            void* out, int out_is_fp32, void* workspace, cudaStream_t stream) {
    const int hq = ctx->cfg.n_q_heads, hkv = ctx->cfg.n_kv_heads;
    const int ms = max_splits_of(max_pages_per_seq);
    float* part_ml = (float*)workspace;
    const size_t ml_bytes = (((size_t)batch * hkv * ms * HG * 2 * 4) + 255) & ~(size_t)255;
    float* part_acc = (float*)((char*)workspace + ml_bytes);
    // with a window only the pages it touches are scanned
    const int scan_pages = window > 0 ? (window + 2 * NOVAKV_PAGE_TOKENS - 1) / NOVAKV_PAGE_TOKENS : max_pages_per_seq;
    const int grid_x = (min(scan_pages, max_pages_per_seq) + BF16_SPLIT_PAGES - 1) / BF16_SPLIT_PAGES;
    dim3 grid(grid_x, hkv, batch);
    {
        novakv_prof_scope ps(ctx, 2, stream);
        novakv_bf16_stage1_kernel<D, HG><<<grid, BF16_WARPS * 32, 0, stream>>>(q, k_pages, v_pages, n_pages, page_table,
            max_pages_per_seq, seq_lens, hq, hkv, sm_scale * 1.4426950408889634f, window, ms, part_ml, part_acc);
        ps.end();
        ctx->launches++;
    }
    novakv_bf16_merge_kernel<D, HG><<<batch * hkv, 256, 0, stream>>>(part_ml, part_acc, seq_lens, max_pages_per_seq, hq, hkv,
                                                                     window, ms, out, out_is_fp32);
    ctx->launches++;
    return cudaGetLastError() == cudaSuccess ? NOVAKV_OK : NOVAKV_ECUDA;
}

}  // namespace

size_t novakv_bf16_ws_bytes(const novakv_ctx* ctx, int batch, int max_pages_per_seq) {
    const int ms = max_splits_of(max_pages_per_seq);
    const size_t n = (size_t)batch * ctx->cfg.n_kv_heads * ms * ctx->hg;
    return ((n * 2 * 4 + 255) & ~(size_t)255) + n * ctx->cfg.head_dim * 4 + 256;
}

novakv_status novakv_launch_bf16_decode(novakv_ctx* ctx, const __nv_bfloat16* q,
    const __nv_bfloat16* k_pages, const __nv_bfloat16* v_pages, int n_pages,
    const int32_t* page_table, int max_pages_per_seq, const int32_t* seq_lens, int batch,
    float sm_scale, int window, void* out, int out_is_fp32, void* workspace, size_t workspace_bytes,
    cudaStream_t stream) {
    (void)workspace_bytes;
    const int d = ctx->cfg.head_dim, hg = ctx->hg;
    if (d == 128 && hg == 4)
        return launch_bf16_t<128, 4>(ctx, q, k_pages, v_pages, n_pages, page_table, max_pages_per_seq, seq_lens, batch,
                                     sm_scale, window, out, out_is_fp32, workspace, stream);
    if (d == 64 && hg == 8)
        return launch_bf16_t<64, 8>(ctx, q, k_pages, v_pages, n_pages, page_table, max_pages_per_seq, seq_lens, batch,
                                    sm_scale, window, out, out_is_fp32, workspace, stream);
    if (d == 64 && hg == 4)
        return launch_bf16_t<64, 4>(ctx, q, k_pages, v_pages, n_pages, page_table, max_pages_per_seq, seq_lens, batch,
                                    sm_scale, window, out, out_is_fp32, workspace, stream);
    return NOVAKV_ESHAPE;      // the comparator covers the benchmarked shapes only
}
