// Host side of the C ABI: context, calibration upload, argument validation, dispatch.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "novakv_internal.cuh"

#define CUDA_OK(expr)                                   \
    do {                                                \
        cudaError_t e__ = (expr);                       \
        if (e__ != cudaSuccess) return NOVAKV_ECUDA;    \
    } while (0)

extern "C" const char* novakv_status_string(novakv_status s) {
    switch (s) {
        case NOVAKV_OK: return "ok";
        case NOVAKV_EINVAL: return "invalid argument";
        case NOVAKV_ESHAPE: return "unsupported shape";
        case NOVAKV_ENOCALIB: return "layer has no calibration";
        case NOVAKV_EPAGE: return "inconsistent page geometry";
        case NOVAKV_EWORKSPACE: return "workspace missing or too small";
        case NOVAKV_ECUDA: return "CUDA runtime error";
        case NOVAKV_EUNSUPPORTED: return "unsupported calibration content";
    }
    return "unknown status";
}

static bool shape_supported(const novakv_config& c) {
    if (c.group_size != NOVAKV_G || c.codebook_size != NOVAKV_C || c.page_tokens != NOVAKV_PAGE_TOKENS) return false;
    if (c.head_dim != 64 && c.head_dim != 128) return false;
    if (c.n_kv_heads <= 0 || c.n_q_heads <= 0 || c.n_q_heads % c.n_kv_heads != 0) return false;
    int hg = c.n_q_heads / c.n_kv_heads;
    if (hg != 1 && hg != 2 && hg != 4 && hg != 8) return false;
    if (c.head_dim == 128 && hg == 8) return false;
    return true;
}

extern "C" novakv_status novakv_create(novakv_ctx** out, const novakv_config* cfg) {
    if (!out || !cfg) return NOVAKV_EINVAL;
    *out = nullptr;
    if (cfg->n_layers <= 0 || cfg->device < 0) return NOVAKV_EINVAL;
    if (!shape_supported(*cfg)) return NOVAKV_ESHAPE;
    int ndev = 0;
    CUDA_OK(cudaGetDeviceCount(&ndev));
    if (cfg->device >= ndev) return NOVAKV_EINVAL;
    CUDA_OK(cudaSetDevice(cfg->device));
    novakv_ctx* ctx = new (std::nothrow) novakv_ctx();
    if (!ctx) return NOVAKV_EINVAL;
    ctx->cfg = *cfg;
    // setting up a segment (score table of 256 x L entries per head) costs about as much as scanning this many pages
    ctx->seg_weight = cfg->head_dim == 128 ? 40 : 24;
    ctx->hg = cfg->n_q_heads / cfg->n_kv_heads;
    ctx->n_groups = cfg->head_dim / NOVAKV_G;
    ctx->layers.resize(cfg->n_layers);
    if (cudaDeviceGetAttribute(&ctx->n_sm, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess ||
        cudaMalloc(&ctx->dev_status, 256) != cudaSuccess ||
        cudaMemset(ctx->dev_status, 0, 256) != cudaSuccess) {
        delete ctx;
        return NOVAKV_ECUDA;
    }
    {
        // product codebook of the scalar INT2 value codec: byte c decodes to the levels (c & 3, (c >> 2) & 3,
        // (c >> 4) & 3, c >> 6), the same for every group and head, in the layout the value gather reads
        // (uint8 [256 codes][32 slots][4])
        const size_t n = (size_t)NOVAKV_C * 32 * NOVAKV_G;
        std::vector<uint8_t> img(n);
        for (size_t i = 0; i < n; ++i) {
            const int comp = (int)(i % NOVAKV_G), code = (int)(i / (32 * NOVAKV_G));
            img[i] = (uint8_t)((code >> (2 * comp)) & 3);
        }
        if (cudaMalloc(&ctx->int2_img, n) != cudaSuccess ||
            cudaMemcpy(ctx->int2_img, img.data(), n, cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaFree(ctx->dev_status);
            cudaFree(ctx->int2_img);
            delete ctx;
            return NOVAKV_ECUDA;
        }
    }
    *out = ctx;
    return NOVAKV_OK;
}

static void free_layer(novakv_layer& ly) {
    cudaFree(ly.rk_d); cudaFree(ly.rv_d); cudaFree(ly.k_mean_d); cudaFree(ly.v_mean_d);
    cudaFree(ly.rk_d_mma); cudaFree(ly.rv_d_mma); cudaFree(ly.k_mean);
    cudaFree(ly.cb_k); cudaFree(ly.cb_v); cudaFree(ly.rk_inv_t); cudaFree(ly.rv_t);
    cudaFree(ly.v_mean); cudaFree(ly.cb_k_lut); cudaFree(ly.cb_v_u8); cudaFree(ly.v_scale); cudaFree(ly.v_off);
    cudaFree(ly.k_mean_eff); cudaFree(ly.k_center);
    ly = novakv_layer();
}

extern "C" novakv_status novakv_destroy(novakv_ctx* ctx) {
    if (!ctx) return NOVAKV_EINVAL;
    cudaSetDevice(ctx->cfg.device);
    cudaDeviceSynchronize();
    for (auto& ly : ctx->layers) free_layer(ly);
    for (int k = 0; k < 3; ++k)
        for (auto& e : ctx->prof[k]) { cudaEventDestroy(e.start); cudaEventDestroy(e.stop); }
    for (auto& e : ctx->prof_free) { cudaEventDestroy(e.start); cudaEventDestroy(e.stop); }
    cudaFree(ctx->dev_status);
    cudaFree(ctx->int2_img);
    delete ctx;
    return NOVAKV_OK;
}

template <typename T>
static cudaError_t upload(T** dst, const std::vector<T>& host) {
    cudaError_t e = cudaMalloc(dst, host.size() * sizeof(T));
    if (e != cudaSuccess) return e;
    return cudaMemcpy(*dst, host.data(), host.size() * sizeof(T), cudaMemcpyHostToDevice);
}

extern "C" novakv_status novakv_load_calibration(novakv_ctx* ctx, int layer, const novakv_calibration* h) {
    if (!ctx || !h || layer < 0 || layer >= ctx->cfg.n_layers) return NOVAKV_EINVAL;
    if (!h->rk || !h->rk_inv_t || !h->rv || !h->cb_k || !h->cb_v) return NOVAKV_EINVAL;
    const int H = ctx->cfg.n_kv_heads, d = ctx->cfg.head_dim, L = ctx->n_groups, C = NOVAKV_C, g = NOVAKV_G;
    const size_t n_mat = (size_t)H * d * d, n_vec = (size_t)H * d, n_cb = (size_t)H * L * C * g;

    // Value codewords: every coordinate (KV head, group l, component i) must lie on its own 7-bit grid
    // lo + u (hi - lo) / 127, u = 0 .. 127, with lo / hi the smallest / largest value that coordinate takes over
    // the 256 codewords (the calibrator snaps them after Lloyd, as the paper snaps its codebooks to a narrow
    // format offline).  The kernel keeps the indices u (4 bytes per codeword, top bit clear: a byte and its
    // replicated top bit form the binary16 number u 2^-24) and applies step and offset once per output
    // coefficient.  The grid is evaluated in binary64 and rounded to binary32 exactly as below.
    std::vector<uint8_t> cbv_u8((size_t)H * C * 32 * g, 0);
    std::vector<float> v_scale((size_t)H * d, 1.f), v_off((size_t)H * d, 0.f);
    for (int hh = 0; hh < H; ++hh)
        for (int l = 0; l < L; ++l)
            for (int i = 0; i < g; ++i) {
                float lo = h->cb_v[(((size_t)hh * L + l) * C) * g + i], hi = lo;
                for (int c = 1; c < C; ++c) {
                    const float x = h->cb_v[(((size_t)hh * L + l) * C + c) * g + i];
                    if (!(x == x)) return NOVAKV_EUNSUPPORTED;
                    lo = x < lo ? x : lo;
                    hi = x > hi ? x : hi;
                }
                double step = ((double)hi - (double)lo) / 127.0;
                if (!(step > 0.0) || !(step < 1e300)) step = 1.0;
                for (int c = 0; c < C; ++c) {
                    const float x = h->cb_v[(((size_t)hh * L + l) * C + c) * g + i];
                    double u = nearbyint(((double)x - (double)lo) / step);
                    if (u < 0.0) u = 0.0;
                    if (u > 127.0) u = 127.0;
                    if ((float)((double)lo + step * u) != x) return NOVAKV_EUNSUPPORTED;
                    cbv_u8[(((size_t)hh * C + c) * 32 + l) * g + i] = (uint8_t)u;
                }
                v_scale[(size_t)hh * d + l * g + i] = (float)step;
                v_off[(size_t)hh * d + l * g + i] = (float)((double)lo + 64.0 * step);
            }

    std::vector<double> rk_d(n_mat), rv_d(n_mat), km_d(n_vec, 0.0), vm_d(n_vec, 0.0);
    std::vector<float> vm_f(n_vec, 0.f), km_f(n_vec, 0.f);
    for (size_t i = 0; i < n_mat; ++i) { rk_d[i] = (double)h->rk[i]; rv_d[i] = (double)h->rv[i]; }
    // the same matrices with the input dimension blocked by 4: img[h][k/4][c][k%4] = R[h][k][c]
    std::vector<double> rk_mma(n_mat), rv_mma(n_mat);
    for (int hh = 0; hh < H; ++hh)
        for (int k = 0; k < d; ++k)
            for (int c = 0; c < d; ++c) {
                const size_t dst = (((size_t)hh * (d / 4) + k / 4) * d + c) * 4 + k % 4, src = ((size_t)hh * d + k) * d + c;
                rk_mma[dst] = rk_d[src];
                rv_mma[dst] = rv_d[src];
            }
    if (h->k_mean) for (size_t i = 0; i < n_vec; ++i) { km_d[i] = (double)h->k_mean[i]; km_f[i] = h->k_mean[i]; }
    if (h->v_mean) for (size_t i = 0; i < n_vec; ++i) { vm_d[i] = (double)h->v_mean[i]; vm_f[i] = h->v_mean[i]; }

    // Key codebook in score-table order [Hkv][code][l][4], centred: every (group, component) has the midrange of
    // its 256 codeword values subtracted, which shrinks the table entries (they are kept in binary16).  The
    // softmax does not see the shift: it moves all logits of a query by the same <q', centre>.
    std::vector<float> cbk_lut((size_t)H * C * L * g), kcen((size_t)H * d, 0.f), km_eff(n_vec, 0.f);
    for (int hh = 0; hh < H; ++hh)
        for (int l = 0; l < L; ++l)
            for (int i = 0; i < g; ++i) {
                float lo = h->cb_k[(((size_t)hh * L + l) * C) * g + i], hi = lo;
                for (int c = 1; c < C; ++c) {
                    const float x = h->cb_k[(((size_t)hh * L + l) * C + c) * g + i];
                    lo = x < lo ? x : lo;
                    hi = x > hi ? x : hi;
                }
                const float cen = (float)(0.5 * ((double)lo + (double)hi));
                kcen[(size_t)hh * d + l * g + i] = cen;
                for (int c = 0; c < C; ++c)
                    cbk_lut[(((size_t)hh * C + c) * L + l) * g + i] =
                        (float)((double)h->cb_k[(((size_t)hh * L + l) * C + c) * g + i] - (double)cen);
            }
    // what the centred table drops from a logit, <q rk_inv_t, centre> = q . (rk_inv_t centre^T), joins q . k_mean
    for (int hh = 0; hh < H; ++hh)
        for (int r = 0; r < d; ++r) {
            double acc = km_d[(size_t)hh * d + r];
            for (int c = 0; c < d; ++c) acc += (double)h->rk_inv_t[((size_t)hh * d + r) * d + c] * (double)kcen[(size_t)hh * d + c];
            km_eff[(size_t)hh * d + r] = (float)acc;
        }

    CUDA_OK(cudaSetDevice(ctx->cfg.device));
    novakv_layer& ly = ctx->layers[layer];
    if (ly.loaded) { cudaDeviceSynchronize(); free_layer(ly); }
    std::vector<float> cbk(h->cb_k, h->cb_k + n_cb), cbv(h->cb_v, h->cb_v + n_cb);
    std::vector<float> rkinv(h->rk_inv_t, h->rk_inv_t + n_mat), rvt(n_mat);
    for (int hh = 0; hh < H; ++hh)       // transposed copy: rv_t[c][r] = rv[r][c], so that o = o' rv^T reads rows
        for (int r = 0; r < d; ++r)
            for (int c = 0; c < d; ++c) rvt[((size_t)hh * d + c) * d + r] = h->rv[((size_t)hh * d + r) * d + c];
    bool ok = upload(&ly.rk_d, rk_d) == cudaSuccess && upload(&ly.rv_d, rv_d) == cudaSuccess &&
              upload(&ly.rk_d_mma, rk_mma) == cudaSuccess && upload(&ly.rv_d_mma, rv_mma) == cudaSuccess &&
              upload(&ly.k_mean_d, km_d) == cudaSuccess && upload(&ly.v_mean_d, vm_d) == cudaSuccess &&
              upload(&ly.cb_k, cbk) == cudaSuccess && upload(&ly.cb_v, cbv) == cudaSuccess &&
              upload(&ly.rk_inv_t, rkinv) == cudaSuccess && upload(&ly.rv_t, rvt) == cudaSuccess &&
              upload(&ly.v_mean, vm_f) == cudaSuccess && upload(&ly.k_mean, km_f) == cudaSuccess && upload(&ly.cb_k_lut, cbk_lut) == cudaSuccess &&
              upload(&ly.cb_v_u8, cbv_u8) == cudaSuccess && upload(&ly.v_scale, v_scale) == cudaSuccess &&
              upload(&ly.v_off, v_off) == cudaSuccess && upload(&ly.k_mean_eff, km_eff) == cudaSuccess &&
              upload(&ly.k_center, kcen) == cudaSuccess;
    if (!ok) { free_layer(ly); return NOVAKV_ECUDA; }
    ly.loaded = true;
    return NOVAKV_OK;
}

extern "C" size_t novakv_page_bytes(const novakv_ctx* ctx) {
    if (!ctx) return 0;
    return (size_t)ctx->cfg.n_kv_heads * NOVAKV_PAGE_TOKENS * ctx->n_groups;
}

extern "C" size_t novakv_decode_workspace_bytes(const novakv_ctx* ctx, int batch) {
    if (!ctx || batch <= 0) return 0;
    return novakv_decode_ws_bytes(ctx, batch);
}

static novakv_status check_common(const novakv_ctx* ctx, int layer) {
    if (!ctx) return NOVAKV_EINVAL;
    if (layer < 0 || layer >= ctx->cfg.n_layers) return NOVAKV_EINVAL;
    if (!ctx->layers[layer].loaded) return NOVAKV_ENOCALIB;
    return NOVAKV_OK;
}

extern "C" novakv_status novakv_encode_append(novakv_ctx* ctx, int layer, const void* k_new,
    const void* v_new, const int32_t* tok_seq, const int32_t* tok_pos, int n_tokens, uint8_t* k_pages,
    uint8_t* v_pages, int n_pages, const int32_t* page_table, int max_pages_per_seq, int n_seq,
    int32_t* seq_lens, novakv_stream stream) {
    novakv_status st = check_common(ctx, layer);
    if (st != NOVAKV_OK) return st;
    if (n_tokens < 0) return NOVAKV_EINVAL;
    if (n_tokens == 0) return NOVAKV_OK;
    if (!k_new || !v_new || !tok_seq || !tok_pos || !k_pages || !v_pages || !page_table || !seq_lens) return NOVAKV_EINVAL;
    if (n_pages <= 0 || max_pages_per_seq <= 0 || n_seq <= 0) return NOVAKV_EPAGE;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return NOVAKV_ECUDA;
    return novakv_launch_encode(ctx, ctx->layers[layer], (const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new,
                                tok_seq, tok_pos, n_tokens, k_pages, v_pages, n_pages, page_table,
                                max_pages_per_seq, n_seq, seq_lens, (cudaStream_t)stream);
}

extern "C" novakv_status novakv_decode_attention(novakv_ctx* ctx, int layer, const void* q,
    const uint8_t* k_pages, const uint8_t* v_pages, int n_pages, const int32_t* page_table,
    int max_pages_per_seq, const int32_t* seq_lens, int batch, float sm_scale, void* out, int out_is_fp32,
    void* workspace, size_t workspace_bytes, novakv_stream stream) {
    novakv_status st = check_common(ctx, layer);
    if (st != NOVAKV_OK) return st;
    if (batch < 0) return NOVAKV_EINVAL;
    if (batch == 0) return NOVAKV_OK;
    if (!q || !k_pages || !v_pages || !page_table || !seq_lens || !out) return NOVAKV_EINVAL;
    if (n_pages <= 0 || max_pages_per_seq <= 0) return NOVAKV_EPAGE;
    if (((uintptr_t)k_pages & 15) || ((uintptr_t)v_pages & 15)) return NOVAKV_EINVAL;   // bulk copies need 16-byte alignment
    if (!(sm_scale == sm_scale)) return NOVAKV_EINVAL;
    if (!workspace || workspace_bytes < novakv_decode_ws_bytes(ctx, batch) || ((uintptr_t)workspace & 255)) return NOVAKV_EWORKSPACE;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return NOVAKV_ECUDA;
    return novakv_launch_decode(ctx, ctx->layers[layer], (const __nv_bfloat16*)q, k_pages, v_pages, n_pages,
                                page_table, max_pages_per_seq, seq_lens, batch, sm_scale, out, out_is_fp32,
                                workspace, workspace_bytes, (cudaStream_t)stream);
}

extern "C" size_t novakv_scale_page_bytes(const novakv_ctx* ctx) {
    return ctx ? (size_t)ctx->cfg.n_kv_heads * NOVAKV_PAGE_TOKENS * 2 : 0;
}

extern "C" novakv_status novakv_encode_append_scaled(novakv_ctx* ctx, int layer, const void* k_new,
    const void* v_new, const int32_t* tok_seq, const int32_t* tok_pos, int n_tokens, uint8_t* k_pages,
    uint8_t* v_pages, void* k_scales, int n_pages, const int32_t* page_table, int max_pages_per_seq, int n_seq,
    int32_t* seq_lens, novakv_stream stream) {
    novakv_status st = check_common(ctx, layer);
    if (st != NOVAKV_OK) return st;
    if (n_tokens < 0) return NOVAKV_EINVAL;
    if (n_tokens == 0) return NOVAKV_OK;
    if (!k_new || !v_new || !tok_seq || !tok_pos || !k_pages || !v_pages || !k_scales || !page_table || !seq_lens) return NOVAKV_EINVAL;
    if (n_pages <= 0 || max_pages_per_seq <= 0 || n_seq <= 0) return NOVAKV_EPAGE;
    if ((uintptr_t)k_scales & 1) return NOVAKV_EINVAL;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return NOVAKV_ECUDA;
    return novakv_launch_encode(ctx, ctx->layers[layer], (const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new,
                                tok_seq, tok_pos, n_tokens, k_pages, v_pages, n_pages, page_table,
                                max_pages_per_seq, n_seq, seq_lens, (cudaStream_t)stream, (__nv_bfloat16*)k_scales);
}

extern "C" novakv_status novakv_decode_attention_scaled(novakv_ctx* ctx, int layer, const void* q,
    const uint8_t* k_pages, const uint8_t* v_pages, const void* k_scales, int n_pages, const int32_t* page_table,
    int max_pages_per_seq, const int32_t* seq_lens, int batch, float sm_scale, void* out, int out_is_fp32,
    void* workspace, size_t workspace_bytes, novakv_stream stream) {
    novakv_status st = check_common(ctx, layer);
    if (st != NOVAKV_OK) return st;
    if (batch < 0) return NOVAKV_EINVAL;
    if (batch == 0) return NOVAKV_OK;
    if (!q || !k_pages || !v_pages || !k_scales || !page_table || !seq_lens || !out) return NOVAKV_EINVAL;
    if (n_pages <= 0 || max_pages_per_seq <= 0) return NOVAKV_EPAGE;
    if (((uintptr_t)k_pages & 15) || ((uintptr_t)v_pages & 15) || ((uintptr_t)k_scales & 1)) return NOVAKV_EINVAL;
    if (!(sm_scale == sm_scale)) return NOVAKV_EINVAL;
    if (!workspace || workspace_bytes < novakv_decode_ws_bytes(ctx, batch) || ((uintptr_t)workspace & 255)) return NOVAKV_EWORKSPACE;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return NOVAKV_ECUDA;
    return novakv_launch_decode(ctx, ctx->layers[layer], (const __nv_bfloat16*)q, k_pages, v_pages, n_pages,
                                page_table, max_pages_per_seq, seq_lens, batch, sm_scale, out, out_is_fp32,
                                workspace, workspace_bytes, (cudaStream_t)stream, (const __nv_bfloat16*)k_scales);
}

extern "C" novakv_status novakv_decode_attention_sink(novakv_ctx* ctx, int layer, const void* q,
    const uint8_t* k_pages, const uint8_t* v_pages, const void* k_scales, const float* sink_logits, int n_pages,
    const int32_t* page_table, int max_pages_per_seq, const int32_t* seq_lens, int batch, float sm_scale, void* out,
    int out_is_fp32, void* workspace, size_t workspace_bytes, novakv_stream stream) {
    novakv_status st = check_common(ctx, layer);
    if (st != NOVAKV_OK) return st;
    if (batch < 0) return NOVAKV_EINVAL;
    if (batch == 0) return NOVAKV_OK;
    if (!q || !k_pages || !v_pages || !sink_logits || !page_table || !seq_lens || !out) return NOVAKV_EINVAL;
    if (n_pages <= 0 || max_pages_per_seq <= 0) return NOVAKV_EPAGE;
    if (((uintptr_t)k_pages & 15) || ((uintptr_t)v_pages & 15) || ((uintptr_t)k_scales & 1) || ((uintptr_t)sink_logits & 3)) return NOVAKV_EINVAL;
    if (!(sm_scale == sm_scale)) return NOVAKV_EINVAL;
    if (!workspace || workspace_bytes < novakv_decode_ws_bytes(ctx, batch) || ((uintptr_t)workspace & 255)) return NOVAKV_EWORKSPACE;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return NOVAKV_ECUDA;
    return novakv_launch_decode(ctx, ctx->layers[layer], (const __nv_bfloat16*)q, k_pages, v_pages, n_pages,
                                page_table, max_pages_per_seq, seq_lens, batch, sm_scale, out, out_is_fp32,
                                workspace, workspace_bytes, (cudaStream_t)stream, (const __nv_bfloat16*)k_scales,
                                sink_logits);
}

extern "C" novakv_status novakv_decode_attention_banded(novakv_ctx* ctx, int layer, const void* q,
    const uint8_t* k_pages, const uint8_t* v_pages, const void* k_scales, const float* sink_logits, int n_pages,
    const int32_t* page_table, int max_pages_per_seq, const int32_t* quant_lens, const void* band_k,
    const void* band_v, int band_cap, int n_sink, const int32_t* band_meta, int batch, float sm_scale, void* out,
    int out_is_fp32, void* workspace, size_t workspace_bytes, novakv_stream stream) {
    novakv_status st = check_common(ctx, layer);
    if (st != NOVAKV_OK) return st;
    if (batch < 0) return NOVAKV_EINVAL;
    if (batch == 0) return NOVAKV_OK;
    if (!q || !k_pages || !v_pages || !page_table || !quant_lens || !band_k || !band_v || !band_meta || !out) return NOVAKV_EINVAL;
    if (n_sink < 0 || n_sink % NOVAKV_PAGE_TOKENS != 0 || band_cap < n_sink) return NOVAKV_EINVAL;
    if (n_pages <= 0 || max_pages_per_seq <= n_sink / NOVAKV_PAGE_TOKENS) return NOVAKV_EPAGE;
    if (((uintptr_t)k_pages & 15) || ((uintptr_t)v_pages & 15) || ((uintptr_t)k_scales & 1) || ((uintptr_t)sink_logits & 3) ||
        ((uintptr_t)band_k & 3) || ((uintptr_t)band_v & 3)) return NOVAKV_EINVAL;
    if (!(sm_scale == sm_scale)) return NOVAKV_EINVAL;
    if (!workspace || workspace_bytes < novakv_decode_ws_bytes(ctx, batch) || ((uintptr_t)workspace & 255)) return NOVAKV_EWORKSPACE;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return NOVAKV_ECUDA;
    novakv_band_args band;
    band.k = (const __nv_bfloat16*)band_k;
    band.v = (const __nv_bfloat16*)band_v;
    band.cap = band_cap;
    band.n_sink = n_sink;
    band.meta = band_meta;
    return novakv_launch_decode(ctx, ctx->layers[layer], (const __nv_bfloat16*)q, k_pages, v_pages, n_pages,
                                page_table, max_pages_per_seq, quant_lens, batch, sm_scale, out, out_is_fp32,
                                workspace, workspace_bytes, (cudaStream_t)stream, (const __nv_bfloat16*)k_scales,
                                sink_logits, &band);
}

extern "C" size_t novakv_value_meta_page_bytes(const novakv_ctx* ctx) {
    return ctx ? (size_t)ctx->cfg.n_kv_heads * NOVAKV_PAGE_TOKENS * 4 : 0;
}

extern "C" novakv_status novakv_encode_append_deployed(novakv_ctx* ctx, int layer, const void* k_new,
    const void* v_new, const int32_t* tok_seq, const int32_t* tok_pos, int n_tokens, uint8_t* k_pages,
    uint8_t* v_pages, void* k_scales, void* v_meta, int n_pages, const int32_t* page_table, int max_pages_per_seq,
    int n_seq, int32_t* seq_lens, novakv_stream stream) {
    novakv_status st = check_common(ctx, layer);
    if (st != NOVAKV_OK) return st;
    if (n_tokens < 0) return NOVAKV_EINVAL;
    if (n_tokens == 0) return NOVAKV_OK;
    if (!k_new || !v_new || !tok_seq || !tok_pos || !k_pages || !v_pages || !k_scales || !v_meta || !page_table || !seq_lens)
        return NOVAKV_EINVAL;
    if (n_pages <= 0 || max_pages_per_seq <= 0 || n_seq <= 0) return NOVAKV_EPAGE;
    if (((uintptr_t)k_scales & 1) || ((uintptr_t)v_meta & 3)) return NOVAKV_EINVAL;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return NOVAKV_ECUDA;
    return novakv_launch_encode(ctx, ctx->layers[layer], (const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new,
                                tok_seq, tok_pos, n_tokens, k_pages, v_pages, n_pages, page_table,
                                max_pages_per_seq, n_seq, seq_lens, (cudaStream_t)stream, (__nv_bfloat16*)k_scales,
                                (__nv_bfloat16*)v_meta);
}

// staging of novakv_band_append: tokens leaving the band [batch * block][Hkv][d] bf16 for K and for V, then the
// (sequence, position) list, each part 256-byte aligned
static size_t band_stage_part(size_t x) { return (x + 255) & ~(size_t)255; }
extern "C" size_t novakv_band_append_staging_bytes(const novakv_ctx* ctx, int batch, int block) {
    if (!ctx || batch <= 0 || block <= 0) return 0;
    const size_t rows = (size_t)batch * block;
    return 2 * band_stage_part(rows * ctx->cfg.n_kv_heads * ctx->cfg.head_dim * 2) + 2 * band_stage_part(rows * 4);
}

extern "C" novakv_status novakv_band_append(novakv_ctx* ctx, int layer, const void* k_new, const void* v_new, int batch,
    void* band_k, void* band_v, int band_cap, int n_sink, int n_rec, int block, int32_t* band_meta, int32_t* quant_lens,
    uint8_t* k_pages, uint8_t* v_pages, void* k_scales, void* v_meta, int n_pages, const int32_t* page_table,
    int max_pages_per_seq, int32_t* seq_lens, void* staging, size_t staging_bytes, novakv_stream stream) {
    novakv_status st = check_common(ctx, layer);
    if (st != NOVAKV_OK) return st;
    if (batch < 0) return NOVAKV_EINVAL;
    if (batch == 0) return NOVAKV_OK;
    if (!k_new || !v_new || !band_k || !band_v || !band_meta || !quant_lens || !k_pages || !v_pages || !page_table || !seq_lens)
        return NOVAKV_EINVAL;
    if (v_meta != nullptr && k_scales == nullptr) return NOVAKV_EUNSUPPORTED;
    if (n_sink < 0 || n_sink % NOVAKV_PAGE_TOKENS != 0 || n_rec <= 0 || block <= 0 || (long)n_sink + n_rec + block > band_cap)
        return NOVAKV_EINVAL;
    if (n_pages <= 0 || max_pages_per_seq <= 0) return NOVAKV_EPAGE;
    if (((uintptr_t)k_new | (uintptr_t)v_new | (uintptr_t)band_k | (uintptr_t)band_v) & 15) return NOVAKV_EINVAL;
    if (!staging || staging_bytes < novakv_band_append_staging_bytes(ctx, batch, block) || ((uintptr_t)staging & 255))
        return NOVAKV_EWORKSPACE;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return NOVAKV_ECUDA;
    const size_t rows = (size_t)batch * block;
    const size_t tok_bytes = band_stage_part(rows * ctx->cfg.n_kv_heads * ctx->cfg.head_dim * 2);
    unsigned char* base = (unsigned char*)staging;
    void* stage_k = base;
    void* stage_v = base + tok_bytes;
    int32_t* tok_seq = (int32_t*)(base + 2 * tok_bytes);
    int32_t* tok_pos = (int32_t*)(base + 2 * tok_bytes + band_stage_part(rows * 4));
    st = novakv_launch_band_insert(ctx, k_new, v_new, batch, band_k, band_v, band_cap, n_sink, n_rec, block, band_meta,
                                   quant_lens, stage_k, stage_v, tok_seq, tok_pos, (cudaStream_t)stream);
    if (st != NOVAKV_OK) return st;
    return novakv_launch_encode(ctx, ctx->layers[layer], (const __nv_bfloat16*)stage_k, (const __nv_bfloat16*)stage_v,
                                tok_seq, tok_pos, (int)rows, k_pages, v_pages, n_pages, page_table, max_pages_per_seq,
                                batch, seq_lens, (cudaStream_t)stream, (__nv_bfloat16*)k_scales, (__nv_bfloat16*)v_meta);
}

extern "C" novakv_status novakv_decode_attention_deployed(novakv_ctx* ctx, int layer, const void* q,
    const uint8_t* k_pages, const uint8_t* v_pages, const void* k_scales, const void* v_meta, const float* sink_logits,
    int n_pages, const int32_t* page_table, int max_pages_per_seq, const int32_t* quant_lens, const void* band_k,
    const void* band_v, int band_cap, int n_sink, const int32_t* band_meta, int batch, float sm_scale, void* out,
    int out_is_fp32, void* workspace, size_t workspace_bytes, novakv_stream stream) {
    novakv_status st = check_common(ctx, layer);
    if (st != NOVAKV_OK) return st;
    if (batch < 0) return NOVAKV_EINVAL;
    if (batch == 0) return NOVAKV_OK;
    if (!q || !k_pages || !v_pages || !k_scales || !v_meta || !page_table || !quant_lens || !out) return NOVAKV_EINVAL;
    const bool banded = band_k != nullptr || band_v != nullptr || band_meta != nullptr;
    if (banded && (!band_k || !band_v || !band_meta)) return NOVAKV_EINVAL;
    if (banded && (n_sink < 0 || n_sink % NOVAKV_PAGE_TOKENS != 0 || band_cap < n_sink)) return NOVAKV_EINVAL;
    if (n_pages <= 0 || max_pages_per_seq <= (banded ? n_sink / NOVAKV_PAGE_TOKENS : 0)) return NOVAKV_EPAGE;
    if (((uintptr_t)k_pages & 15) || ((uintptr_t)v_pages & 15) || ((uintptr_t)k_scales & 1) || ((uintptr_t)v_meta & 3) ||
        ((uintptr_t)sink_logits & 3) || ((uintptr_t)band_k & 3) || ((uintptr_t)band_v & 3)) return NOVAKV_EINVAL;
    if (!(sm_scale == sm_scale)) return NOVAKV_EINVAL;
    if (!workspace || workspace_bytes < novakv_decode_ws_bytes(ctx, batch) || ((uintptr_t)workspace & 255)) return NOVAKV_EWORKSPACE;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return NOVAKV_ECUDA;
    novakv_band_args band;
    band.k = (const __nv_bfloat16*)band_k;
    band.v = (const __nv_bfloat16*)band_v;
    band.cap = band_cap;
    band.n_sink = n_sink;
    band.meta = band_meta;
    return novakv_launch_decode(ctx, ctx->layers[layer], (const __nv_bfloat16*)q, k_pages, v_pages, n_pages,
                                page_table, max_pages_per_seq, quant_lens, batch, sm_scale, out, out_is_fp32,
                                workspace, workspace_bytes, (cudaStream_t)stream, (const __nv_bfloat16*)k_scales,
                                sink_logits, banded ? &band : nullptr, (const __nv_bfloat16*)v_meta);
}

extern "C" novakv_status novakv_last_device_status(novakv_ctx* ctx, novakv_stream stream, uint32_t* word) {
    if (!ctx || !word) return NOVAKV_EINVAL;
    cudaStream_t s = (cudaStream_t)stream;
    CUDA_OK(cudaSetDevice(ctx->cfg.device));
    CUDA_OK(cudaMemcpyAsync(word, ctx->dev_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    CUDA_OK(cudaMemsetAsync(ctx->dev_status, 0, sizeof(uint32_t), s));
    CUDA_OK(cudaStreamSynchronize(s));
    return NOVAKV_OK;
}

// ------------------------------------------------------------------ host-buffer step
static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

extern "C" size_t novakv_step_staging_bytes(const novakv_ctx* ctx, int batch, int n_tokens) {
    if (!ctx || batch < 0 || n_tokens < 0) return 0;
    const size_t d = ctx->cfg.head_dim;
    size_t kv = align256((size_t)n_tokens * ctx->cfg.n_kv_heads * d * 2);
    size_t tok = align256((size_t)n_tokens * 4);
    size_t q = align256((size_t)batch * ctx->cfg.n_q_heads * d * 2);
    size_t o = align256((size_t)batch * ctx->cfg.n_q_heads * d * 4);
    return 2 * kv + 2 * tok + q + o + 256;
}

extern "C" novakv_status novakv_step_host_async(novakv_ctx* ctx, int layer, const void* k_new_host,
    const void* v_new_host, const int32_t* tok_seq_host, const int32_t* tok_pos_host, int n_tokens,
    const void* q_host, uint8_t* k_pages, uint8_t* v_pages, int n_pages, const int32_t* page_table,
    int max_pages_per_seq, int32_t* seq_lens, int batch, float sm_scale, float* out_host, void* staging,
    size_t staging_bytes, void* workspace, size_t workspace_bytes, novakv_stream stream) {
    novakv_status st = check_common(ctx, layer);
    if (st != NOVAKV_OK) return st;
    if (batch <= 0 || n_tokens < 0 || !q_host || !out_host || !staging) return NOVAKV_EINVAL;
    if (n_tokens > 0 && (!k_new_host || !v_new_host || !tok_seq_host || !tok_pos_host)) return NOVAKV_EINVAL;
    if (!k_pages || !v_pages || !page_table || !seq_lens) return NOVAKV_EINVAL;
    if (n_pages <= 0 || max_pages_per_seq <= 0) return NOVAKV_EPAGE;
    if (staging_bytes < novakv_step_staging_bytes(ctx, batch, n_tokens) || ((uintptr_t)staging & 255)) return NOVAKV_EWORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    CUDA_OK(cudaSetDevice(ctx->cfg.device));
    const size_t d = ctx->cfg.head_dim;
    const size_t kv_b = (size_t)n_tokens * ctx->cfg.n_kv_heads * d * 2, tok_b = (size_t)n_tokens * 4;
    const size_t q_b = (size_t)batch * ctx->cfg.n_q_heads * d * 2, o_b = (size_t)batch * ctx->cfg.n_q_heads * d * 4;
    char* p = (char*)staging;
    char* dk = p; p += align256(kv_b);
    char* dv = p; p += align256(kv_b);
    char* dseq = p; p += align256(tok_b);
    char* dpos = p; p += align256(tok_b);
    char* dq = p; p += align256(q_b);
    char* dout = p;
    // Page-locked host buffers are visible to the device under unified addressing: one small kernel pulls
    // all of the step's inputs across the bus (every byte once, coalesced) into `staging`, instead of five
    // copy-engine operations queued one after the other; the merge kernel writes the output straight into
    // the page-locked output buffer.  A buffer that is not page-locked (or not mapped, or not 4-byte
    // aligned) is staged with an asynchronous copy instead.
    auto device_view = [](const void* host_ptr) -> const void* {
        cudaPointerAttributes at;
        if (cudaPointerGetAttributes(&at, host_ptr) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        return (at.type == cudaMemoryTypeHost && at.devicePointer != nullptr) ? at.devicePointer : nullptr;
    };
    novakv_stage_args sa;
    sa.n = 0;
    auto stage_in = [&](const void* host_ptr, char* dev_buf, size_t bytes) -> cudaError_t {
        const void* view = device_view(host_ptr);
        if (view != nullptr && ((uintptr_t)view & 3) == 0 && (bytes & 3) == 0) {
            sa.src[sa.n] = (const uint32_t*)view;
            sa.dst[sa.n] = (uint32_t*)dev_buf;
            sa.words[sa.n] = (unsigned)(bytes / 4);
            ++sa.n;
            return cudaSuccess;
        }
        return cudaMemcpyAsync(dev_buf, host_ptr, bytes, cudaMemcpyHostToDevice, s);
    };
    if (n_tokens > 0) {
        CUDA_OK(stage_in(k_new_host, dk, kv_b));
        CUDA_OK(stage_in(v_new_host, dv, kv_b));
        CUDA_OK(stage_in(tok_seq_host, dseq, tok_b));
        CUDA_OK(stage_in(tok_pos_host, dpos, tok_b));
    }
    CUDA_OK(stage_in(q_host, dq, q_b));
    if (sa.n > 0) {
        if (novakv_launch_stage(ctx, sa, s) != NOVAKV_OK) return NOVAKV_ECUDA;
    }
    const void *uk = dk, *uv = dv, *useq = dseq, *upos = dpos, *uq = dq;
    void* uout = const_cast<void*>(device_view(out_host));
    const bool out_direct = uout != nullptr;
    if (!out_direct) uout = dout;
    if (n_tokens > 0) {
        st = novakv_encode_append(ctx, layer, uk, uv, (const int32_t*)useq, (const int32_t*)upos, n_tokens,
                                  k_pages, v_pages, n_pages, page_table, max_pages_per_seq, batch, seq_lens, stream);
        if (st != NOVAKV_OK) return st;
    }
    st = novakv_decode_attention(ctx, layer, uq, k_pages, v_pages, n_pages, page_table, max_pages_per_seq,
                                 seq_lens, batch, sm_scale, uout, 1, workspace, workspace_bytes, stream);
    if (st != NOVAKV_OK) return st;
    if (!out_direct) CUDA_OK(cudaMemcpyAsync(out_host, dout, o_b, cudaMemcpyDeviceToHost, s));
    return NOVAKV_OK;
}

extern "C" novakv_status novakv_step_host(novakv_ctx* ctx, int layer, const void* k_new_host,
    const void* v_new_host, const int32_t* tok_seq_host, const int32_t* tok_pos_host, int n_tokens,
    const void* q_host, uint8_t* k_pages, uint8_t* v_pages, int n_pages, const int32_t* page_table,
    int max_pages_per_seq, int32_t* seq_lens, int batch, float sm_scale, float* out_host, void* staging,
    size_t staging_bytes, void* workspace, size_t workspace_bytes, novakv_stream stream) {
    const novakv_status st = novakv_step_host_async(ctx, layer, k_new_host, v_new_host, tok_seq_host, tok_pos_host, n_tokens,
                                                    q_host, k_pages, v_pages, n_pages, page_table, max_pages_per_seq, seq_lens,
                                                    batch, sm_scale, out_host, staging, staging_bytes, workspace, workspace_bytes,
                                                    stream);
    if (st != NOVAKV_OK) return st;
    CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
    return NOVAKV_OK;
}

// ------------------------------------------------------------------ helpers for tests / bench
extern "C" novakv_status novakv_search_coefficients(novakv_ctx* ctx, int layer, int which, const float* coef,
    int n, uint8_t* idx_out, novakv_stream stream) {
    novakv_status st = check_common(ctx, layer);
    if (st != NOVAKV_OK) return st;
    if (n < 0 || (which != 0 && which != 1)) return NOVAKV_EINVAL;
    if (n == 0) return NOVAKV_OK;
    if (!coef || !idx_out) return NOVAKV_EINVAL;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return NOVAKV_ECUDA;
    return novakv_launch_search(ctx, ctx->layers[layer], which, coef, n, idx_out, (cudaStream_t)stream);
}

extern "C" size_t novakv_bf16_workspace_bytes(const novakv_ctx* ctx, int batch, int max_pages_per_seq) {
    if (!ctx || batch <= 0 || max_pages_per_seq <= 0) return 0;
    return novakv_bf16_ws_bytes(ctx, batch, max_pages_per_seq);
}

extern "C" novakv_status novakv_bf16_decode_attention(novakv_ctx* ctx, const void* q, const void* k_pages_bf16,
    const void* v_pages_bf16, int n_pages, const int32_t* page_table, int max_pages_per_seq,
    const int32_t* seq_lens, int batch, float sm_scale, int window, void* out, int out_is_fp32,
    void* workspace, size_t workspace_bytes, novakv_stream stream) {
    if (!ctx) return NOVAKV_EINVAL;
    if (batch < 0 || window < 0) return NOVAKV_EINVAL;
    if (batch == 0) return NOVAKV_OK;
    if (!q || !k_pages_bf16 || !v_pages_bf16 || !page_table || !seq_lens || !out) return NOVAKV_EINVAL;
    if (n_pages <= 0 || max_pages_per_seq <= 0) return NOVAKV_EPAGE;
    if (!workspace || workspace_bytes < novakv_bf16_ws_bytes(ctx, batch, max_pages_per_seq) || ((uintptr_t)workspace & 255)) return NOVAKV_EWORKSPACE;
    if (cudaSetDevice(ctx->cfg.device) != cudaSuccess) return NOVAKV_ECUDA;
    return novakv_launch_bf16_decode(ctx, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k_pages_bf16,
                                     (const __nv_bfloat16*)v_pages_bf16, n_pages, page_table, max_pages_per_seq,
                                     seq_lens, batch, sm_scale, window, out, out_is_fp32, workspace,
                                     workspace_bytes, (cudaStream_t)stream);
}

// ------------------------------------------------------------------ profiling
novakv_prof_scope::novakv_prof_scope(novakv_ctx* c, int k, cudaStream_t s) : ctx(c), kind(k), stream(s), active(false) {
    if (!ctx->profile) return;
    if (!ctx->prof_free.empty()) {
        ev = ctx->prof_free.back();
        ctx->prof_free.pop_back();
    } else {
        if (cudaEventCreate(&ev.start) != cudaSuccess) return;
        if (cudaEventCreate(&ev.stop) != cudaSuccess) { cudaEventDestroy(ev.start); return; }
    }
    cudaEventRecord(ev.start, stream);
    active = true;
}

void novakv_prof_scope::end() {
    if (!active) return;
    cudaEventRecord(ev.stop, stream);
    ctx->prof[kind].push_back(ev);
    active = false;
}

extern "C" novakv_status novakv_profile_enable(novakv_ctx* ctx, int on) {
    if (!ctx) return NOVAKV_EINVAL;
    ctx->profile = on != 0;
    return NOVAKV_OK;
}

extern "C" novakv_status novakv_profile_read(novakv_ctx* ctx, int kind, double* total_ms, long* launches) {
    if (!ctx || kind < 0 || kind > 2 || !total_ms || !launches) return NOVAKV_EINVAL;
    CUDA_OK(cudaSetDevice(ctx->cfg.device));
    double tot = 0.0;
    long n = 0;
    for (auto& e : ctx->prof[kind]) {
        CUDA_OK(cudaEventSynchronize(e.stop));
        float ms = 0.f;
        CUDA_OK(cudaEventElapsedTime(&ms, e.start, e.stop));
        tot += ms;
        n++;
        ctx->prof_free.push_back(e);
    }
    ctx->prof[kind].clear();
    *total_ms = tot;
    *launches = n;
    return NOVAKV_OK;
}

extern "C" novakv_status novakv_debug_set_scan_ctas(novakv_ctx* ctx, int n_ctas) {
    if (!ctx || n_ctas < 0) return NOVAKV_EINVAL;
    ctx->scan_ctas = n_ctas;
    return NOVAKV_OK;
}

extern "C" novakv_status novakv_debug_set_segment_weight(novakv_ctx* ctx, int pages) {
    if (!ctx || pages < 0 || pages > 4096) return NOVAKV_EINVAL;
    ctx->seg_weight = pages;
    return NOVAKV_OK;
}

extern "C" novakv_status novakv_debug_set_fused_merge(novakv_ctx* ctx, int on) {
    if (!ctx || (on != 0 && on != 1)) return NOVAKV_EINVAL;
    ctx->fused_merge = on != 0;
    return NOVAKV_OK;
}

extern "C" novakv_status novakv_debug_set_value_path(novakv_ctx* ctx, int path) {
    if (!ctx || (path != 0 && path != 1)) return NOVAKV_EINVAL;
    ctx->value_path = path;
    return NOVAKV_OK;
}

extern "C" long novakv_launch_count(const novakv_ctx* ctx) { return ctx ? ctx->launches : 0; }
