// Write path: forward transforms (binary64) + brute-force nearest-codeword search + paged store.
// One CTA handles a tile of tokens for one (KV head, side); side 0 = keys, 1 = values.
//
// The search is ALU-bound (256 distance evaluations per group, per token, per side); the codebook
// of the CTA's head and side stays in shared memory and every warp reads codewords as broadcasts.
//
// The index the write path stores is the exact Euclidean nearest codeword of the binary64 coefficient
// (lowest index on a tie).  The 256 distances are evaluated in binary32; beside the minimum the search
// keeps the second smallest distance, and whenever the two are closer than a rigorous bound on what the
// binary32 evaluation (coefficient rounding included) can have moved them, the group is searched again in
// binary64 by the whole warp (certified search).  The binary32 result is kept only where it provably
// equals the binary64 one.
#include <math_constants.h>
#ifdef NOVAKV_TIMING
#include <cstdio>
#endif

#include <cooperative_groups.h>

#include "novakv_internal.cuh"

namespace {

constexpr int ENC_THREADS = 512;
constexpr int ENC_TILE = 64;   // tokens per tile (search granularity)
#ifndef NOVAKV_SMALL_APPEND_TOKENS
#define NOVAKV_SMALL_APPEND_TOKENS 256   // batches up to this size take the per-group append kernel
#endif

// Shared-memory plan of the search-only kernel: codebook, one tile of coefficients, its indices.
template <int D>
struct EncSmem {
    static constexpr int L = D / NOVAKV_G;
    static constexpr int RSTRIDE = D + 4;                       // floats; keeps 128-bit row reads conflict-free
    static constexpr size_t cb_bytes = (size_t)L * NOVAKV_C * NOVAKV_G * sizeof(float);
    static constexpr size_t r_bytes = (size_t)ENC_TILE * RSTRIDE * sizeof(float);
    static constexpr size_t idx_bytes = (size_t)ENC_TILE * L;
    static constexpr size_t total = cb_bytes + r_bytes + idx_bytes;
};

#ifdef NOVAKV_SCALAR_SEARCH
// Scalar form of the binary32 distance: fma(e3,e3,fma(e2,e2,fma(e1,e1,e0*e0))).
__device__ __forceinline__ float dist4(const float4 r, const float4 c) {
    const float e0 = __fsub_rn(r.x, c.x), e1 = __fsub_rn(r.y, c.y);
    const float e2 = __fsub_rn(r.z, c.z), e3 = __fsub_rn(r.w, c.w);
    return __fmaf_rn(e3, e3, __fmaf_rn(e2, e2, __fmaf_rn(e1, e1, __fmul_rn(e0, e0))));
}
#endif

// Packed binary32 pairs: two IEEE operations per instruction (same roundings as the scalar forms).
__device__ __forceinline__ uint64_t pk2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1,%2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// Distances of one coefficient vector (each component duplicated into a pair) to two codewords at once:
// cw[i] = (codeword c, component i ; codeword c+1, component i).  Same chain as dist4, per half.
__device__ __forceinline__ void dist4x2(const uint64_t (&r2)[4], const uint64_t (&cw)[4], float& d0, float& d1) {
#ifdef NOVAKV_SCALAR_SEARCH
    float r[4], lo[4], hi[4], dummy;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        asm("mov.b64 {%0,%1}, %2;" : "=f"(r[i]), "=f"(dummy) : "l"(r2[i]));
        asm("mov.b64 {%0,%1}, %2;" : "=f"(lo[i]), "=f"(hi[i]) : "l"(cw[i]));
    }
    d0 = dist4(make_float4(r[0], r[1], r[2], r[3]), make_float4(lo[0], lo[1], lo[2], lo[3]));
    d1 = dist4(make_float4(r[0], r[1], r[2], r[3]), make_float4(hi[0], hi[1], hi[2], hi[3]));
#else
    const uint64_t e0 = sub2(r2[0], cw[0]), e1 = sub2(r2[1], cw[1]), e2 = sub2(r2[2], cw[2]), e3 = sub2(r2[3], cw[3]);
    const uint64_t d = fma2(e3, e3, fma2(e2, e2, fma2(e1, e1, mul2(e0, e0))));
    asm("mov.b64 {%0,%1}, %2;" : "=f"(d0), "=f"(d1) : "l"(d));
#endif
}

// Shared-memory image of a (head, side) codebook for the search: [L][128 codeword pairs][4 components][2].
__device__ __forceinline__ void fill_codebook_pairs(float* cb_s, const float4* __restrict__ cb_g, int n_groups) {
    for (int i = threadIdx.x; i < n_groups * NOVAKV_C; i += ENC_THREADS) {
        const float4 v = cb_g[i];
        float* dst = cb_s + (size_t)(i >> 1) * 8 + (i & 1);
        dst[0] = v.x; dst[2] = v.y; dst[4] = v.z; dst[6] = v.w;
    }
}

__device__ __forceinline__ float fmin3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Warp-cooperative exact search of one (token, group) in binary64: all 32 lanes call it with the same
// arguments and get the same result.  The coefficient is either taken from shared memory (EXACT_IN_SMEM:
// the binary32 values there ARE the vector to encode: given coefficients, normalised keys) or recomputed in
// binary64 from the token's bfloat16 input row and the transform's columns 4l .. 4l+3.  Lane i evaluates the
// codewords i, i+32, ... in ascending order with a strict '<'; the warp then keeps the smallest distance
// and, among equal distances, the lowest index.
template <int D, bool EXACT_IN_SMEM>
__device__ __noinline__ int exact_search_group(const float* r_row_s, const __nv_bfloat16* __restrict__ x_row_g,
                                               const double* mean_s, const double* __restrict__ R_plain /* [D][D] */,
                                               int l, const float* cb_pairs_s /* [L][128][4][2] */) {
    const int lane = threadIdx.x & 31;
    double r[4];
    if (EXACT_IN_SMEM) {
#pragma unroll
        for (int c = 0; c < 4; ++c) r[c] = (double)r_row_s[l * 4 + c];
    } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) r[c] = 0.0;
        for (int k = lane; k < D; k += 32) {
            const double xc = (double)__bfloat162float(x_row_g[k]) - mean_s[k];
            const double2 r01 = *reinterpret_cast<const double2*>(R_plain + (size_t)k * D + l * 4);
            const double2 r23 = *reinterpret_cast<const double2*>(R_plain + (size_t)k * D + l * 4 + 2);
            r[0] = fma(xc, r01.x, r[0]); r[1] = fma(xc, r01.y, r[1]);
            r[2] = fma(xc, r23.x, r[2]); r[3] = fma(xc, r23.y, r[3]);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) r[c] += __shfl_xor_sync(0xffffffffu, r[c], o);
    }
    double best = CUDART_INF;
    int bi = lane;
    const float* cb = cb_pairs_s + (size_t)l * NOVAKV_C * 4;
#pragma unroll
    for (int j = 0; j < NOVAKV_C / 32; ++j) {
        const int code = lane + 32 * j;
        const float* cw = cb + (size_t)(code >> 1) * 8 + (code & 1);
        double dd = 0.0;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const double e = r[c] - (double)cw[2 * c];
            dd = __dadd_rn(dd, __dmul_rn(e, e));
        }
        if (dd < best) { best = dd; bi = code; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ob < best || (ob == best && oi < bi)) { best = ob; bi = oi; }
    }
    return bi;
}

// What the binary32 evaluation can have moved a squared distance by: the coefficient vector of the group
// is off by at most delta in norm (its rounding to binary32), the eight operations of the distance add a
// relative 6 * 2^-24.  |d32 - d| <= 2 sqrt(d) delta + delta^2 + 6 * 2^-24 d; the test below uses twice the
// bound at the larger of the two distances (both have moved) with some slack on the constants.
__device__ __forceinline__ bool needs_exact_search(float best, float second, float delta) {
    const float thr = 4.5f * sqrtf(second) * delta + 2.5f * delta * delta + 9.6e-7f * second;     // 9.6e-7 > 16 * 2^-24
    return !(second - best > thr);
}

// Search of the tile's coefficients (r_s, [ENC_TILE][RSTRIDE] float) against the paired codebook image.
// Warp w of n_warps owns groups w, w+n_warps, ...; lane t owns tokens t and t+32.
// The binary32 pass finds the first minimum in ascending codeword order (what a scan with a strict '<' keeps)
// in two steps that need far fewer compare/select instructions than a per-codeword running argmin:
//   1. blocks of 8 codewords: the block minimum (a tree of 3-input minima) updates the running minimum with a
//      strict '<', which keeps the first block that attains the overall minimum; the second smallest block
//      minimum is tracked beside it (two more min/max per block);
//   2. the 8 distances of that block are recomputed (same instructions, same bits); the first one equal to
//      the minimum gives the index and the others enter the second smallest distance.
// Then the certification: a group whose two smallest distances are too close to tell apart in binary32 is
// searched again in binary64 by the whole warp (exact_search_group).
// EXACT_IN_SMEM: the binary32 coefficients in r_s are the vector to encode (delta = 0); otherwise they are
// roundings of binary64 coefficients that exact_search_group recomputes from the inputs x_tile_g
// (bfloat16 rows of the tile's tokens, row stride x_stride elements).
template <int D, bool EXACT_IN_SMEM>
__device__ __forceinline__ void search_tile(const float* r_s, const float4* cb_s, uint8_t* idx_s, int n_valid,
                                            int warp, int n_warps, const __nv_bfloat16* __restrict__ x_tile_g,
                                            size_t x_stride, const double* mean_s,
                                            const double* __restrict__ R_plain) {
    constexpr int L = D / NOVAKV_G;
    constexpr int RS = EncSmem<D>::RSTRIDE;
    const int lane = threadIdx.x & 31;
    for (int l = warp; l < L; l += n_warps) {
        const float4 ra = *reinterpret_cast<const float4*>(r_s + (size_t)lane * RS + l * 4);
        const float4 rb = *reinterpret_cast<const float4*>(r_s + (size_t)(lane + 32) * RS + l * 4);
        const uint64_t ra2[4] = {pk2(ra.x, ra.x), pk2(ra.y, ra.y), pk2(ra.z, ra.z), pk2(ra.w, ra.w)};
        const uint64_t rb2[4] = {pk2(rb.x, rb.x), pk2(rb.y, rb.y), pk2(rb.z, rb.z), pk2(rb.w, rb.w)};
        float best_a = CUDART_INF_F, best_b = CUDART_INF_F, sec_a = CUDART_INF_F, sec_b = CUDART_INF_F;
        int blk_a = 0, blk_b = 0;
        const ulonglong2* cb = reinterpret_cast<const ulonglong2*>(cb_s) + (size_t)l * NOVAKV_C;   // 2 x 16 B per pair
#pragma unroll 4
        for (int blk = 0; blk < NOVAKV_C / 8; ++blk) {
            float da[8], db[8];
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                const ulonglong2 q0 = cb[8 * blk + 2 * p], q1 = cb[8 * blk + 2 * p + 1];
                const uint64_t cw[4] = {q0.x, q0.y, q1.x, q1.y};
                dist4x2(ra2, cw, da[2 * p], da[2 * p + 1]);
                dist4x2(rb2, cw, db[2 * p], db[2 * p + 1]);
            }
            const float ma = fmin3(fmin3(da[0], da[1], da[2]), fmin3(da[3], da[4], da[5]), fminf(da[6], da[7]));
            const float mb = fmin3(fmin3(db[0], db[1], db[2]), fmin3(db[3], db[4], db[5]), fminf(db[6], db[7]));
            sec_a = fminf(sec_a, fmaxf(best_a, ma));
            sec_b = fminf(sec_b, fmaxf(best_b, mb));
            if (ma < best_a) { best_a = ma; blk_a = blk; }
            if (mb < best_b) { best_b = mb; blk_b = blk; }
        }
        // the winning blocks again: first codeword whose distance equals the minimum; the block's other
        // distances compete for the second place
        int ia = 8 * blk_a, ib = 8 * blk_b;
        {
            float da[8], db[8];
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                const ulonglong2 qa0 = cb[8 * blk_a + 2 * p], qa1 = cb[8 * blk_a + 2 * p + 1];
                const uint64_t cwa[4] = {qa0.x, qa0.y, qa1.x, qa1.y};
                dist4x2(ra2, cwa, da[2 * p], da[2 * p + 1]);
                const ulonglong2 qb0 = cb[8 * blk_b + 2 * p], qb1 = cb[8 * blk_b + 2 * p + 1];
                const uint64_t cwb[4] = {qb0.x, qb0.y, qb1.x, qb1.y};
                dist4x2(rb2, cwb, db[2 * p], db[2 * p + 1]);
            }
            int ka = 0, kb = 0;
#pragma unroll
            for (int k = 7; k >= 0; --k) {
                if (da[k] == best_a) ka = k;
                if (db[k] == best_b) kb = k;
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                if (k != ka) sec_a = fminf(sec_a, da[k]);
                if (k != kb) sec_b = fminf(sec_b, db[k]);
            }
            ia += ka; ib += kb;
        }
        // certification
        float del_a = 0.f, del_b = 0.f;
        if (!EXACT_IN_SMEM) {
            // |coefficient - its binary32 rounding| <= 2^-24 |coefficient| per component
            del_a = 5.97e-8f * sqrtf(fmaf(ra.x, ra.x, fmaf(ra.y, ra.y, fmaf(ra.z, ra.z, ra.w * ra.w)))) * 1.0001f;
            del_b = 5.97e-8f * sqrtf(fmaf(rb.x, rb.x, fmaf(rb.y, rb.y, fmaf(rb.z, rb.z, rb.w * rb.w)))) * 1.0001f;
        }
        const bool ta = lane < n_valid && needs_exact_search(best_a, sec_a, del_a);
        const bool tb = lane + 32 < n_valid && needs_exact_search(best_b, sec_b, del_b);
        unsigned todo_a = __ballot_sync(0xffffffffu, ta), todo_b = __ballot_sync(0xffffffffu, tb);
        while (todo_a) {
            const int src = __ffs(todo_a) - 1;
            todo_a &= todo_a - 1;
            const int res = exact_search_group<D, EXACT_IN_SMEM>(r_s + (size_t)src * RS, x_tile_g + (size_t)src * x_stride,
                                                                 mean_s, R_plain, l, reinterpret_cast<const float*>(cb_s));
            if (lane == src) ia = res;
        }
        while (todo_b) {
            const int src = __ffs(todo_b) - 1;
            todo_b &= todo_b - 1;
            const int res = exact_search_group<D, EXACT_IN_SMEM>(r_s + (size_t)(src + 32) * RS,
                                                                 x_tile_g + (size_t)(src + 32) * x_stride, mean_s, R_plain, l,
                                                                 reinterpret_cast<const float*>(cb_s));
            if (lane == src) ib = res;
        }
        if (lane < n_valid) idx_s[lane * L + l] = (uint8_t)ia;
        if (lane + 32 < n_valid) idx_s[(lane + 32) * L + l] = (uint8_t)ib;
    }
}

// Named barriers of the tiled encode kernel (hardware barriers; bar.arrive does not block).
__device__ __forceinline__ void nbar_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ __forceinline__ void nbar_arrive(int id, int n) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(n) : "memory"); }
constexpr int BAR_T = 1, BAR_S = 2, BAR_FULL = 3 /* +buf */, BAR_EMPTY = 5 /* +buf */;
constexpr int ENC_HALF_THREADS = ENC_THREADS / 2;

// Shared-memory plan of the pipelined encode kernel.
template <int D>
struct EncPipe {
    static constexpr int L = D / NOVAKV_G;
    static constexpr int RS = D + 4;
    static constexpr int KS = 8;                               // rows of the transform matrix per slab
    static constexpr size_t cb_bytes = (size_t)L * NOVAKV_C * NOVAKV_G * sizeof(float);
    static constexpr size_t r_bytes = (size_t)ENC_TILE * RS * sizeof(float);       // one buffer
    static constexpr size_t slab_x_bytes = (size_t)ENC_TILE * KS * sizeof(double);  // centred inputs [64][KS]
    static constexpr size_t slab_r_bytes = (size_t)KS * D * sizeof(double);         // KS rows of R
    static constexpr size_t slab_bytes = slab_x_bytes + slab_r_bytes;
    static constexpr size_t idx_bytes = (size_t)ENC_TILE * L;
    static constexpr size_t off_r = cb_bytes;
    static constexpr size_t off_slab = off_r + 2 * r_bytes;                         // 2 slab buffers
    static constexpr size_t off_idx = off_slab + 2 * slab_bytes;
    static constexpr size_t off_pos = off_idx + idx_bytes;                          // [2][2][ENC_TILE] ints
    static constexpr size_t off_mean = off_pos + 4 * ENC_TILE * sizeof(int);        // [D] doubles
    static constexpr size_t off_rho = off_mean + D * sizeof(double);                // [2][2][ENC_TILE] floats (key scale | value scale, zero)
    static constexpr size_t total = off_rho + 4 * ENC_TILE * sizeof(float);
    static_assert(total <= 232448, "shared memory budget");
};

// Tiled (prefill) encode, one CTA per (run of 64-token tiles, KV head, side), the codebook of the
// (head, side) resident in shared memory.  The two phases of a tile use different units of the SM:
// the binary64 transform runs on the fp64 pipe and the load/store unit, the 256-way search on the FMA
// pipe.  Half of the warps therefore transform tile i+1 while the other half searches tile i
// (coefficients double-buffered in shared memory, hand-over by named hardware barriers).
// KSC (key format with a per-token scale, Algorithm 3 "Normalize"): after the key transform of a tile
// the transform warps compute rho = ||r||_2 / sqrt(d) of each token's binary32 coefficients (sum of squares
// in binary64), round it to binary32 and then to bfloat16 (a scale that is not positive and finite becomes
// 1), divide the coefficients by it in binary32 (IEEE division) and hand rho to the search warps, which
// store it beside the indices (k_scales [n_pages][Hkv][64]).  Values are not scaled.
// VSQ (scalar INT2 value codec of the deployed format): after the value transform of a tile the transform
// warps form zero = bf16(min) and scale = bf16((max - zero) / 3) per token, replace each coefficient by its
// level clamp(rint((s - zero) / scale), 0, 3), and the other warps pack four levels per byte (the byte of a
// group) instead of searching; (scale, zero) go to v_meta [n_pages][Hkv][64][2].
// FMT: 0 = 2-bit keys and values (vector quantised), 1 = KSC, 2 = KSC and VSQ.
template <int D, int FMT>
__global__ void __launch_bounds__(ENC_THREADS, 1)
novakv_encode_kernel(const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new,
                     const int32_t* __restrict__ tok_seq, const int32_t* __restrict__ tok_pos, int n_tokens,
                     const double* __restrict__ rk_d, const double* __restrict__ rv_d,
                     const double* __restrict__ rk_plain, const double* __restrict__ rv_plain,
                     const double* __restrict__ k_mean_d, const double* __restrict__ v_mean_d,
                     const float* __restrict__ cb_k, const float* __restrict__ cb_v,
                     uint8_t* __restrict__ k_pages, uint8_t* __restrict__ v_pages,
                     __nv_bfloat16* __restrict__ k_scales, __nv_bfloat16* __restrict__ v_meta, int n_pages,
                     const int32_t* __restrict__ page_table, int max_pages_per_seq, int n_seq,
                     int32_t* __restrict__ seq_lens, int n_kv_heads, int tiles_per_cta_k, int tiles_per_cta_v,
                     uint32_t* __restrict__ dev_status) {
    // rk_d / rv_d: the transforms in tensor-core fragment order [d/4][d][4]; rk_plain / rv_plain: the same
    // matrices row-major [d][d] (read only by the certified search's binary64 recomputation)
    constexpr bool KSC = FMT >= 1, VSQ = FMT == 2;
    using P = EncPipe<D>;
    constexpr int L = D / NOVAKV_G, RS = P::RS, NT = ENC_HALF_THREADS;
    extern __shared__ __align__(16) unsigned char smem[];
    float4* cb_s = reinterpret_cast<float4*>(smem);
    uint8_t* idx_s = smem + P::off_idx;
    int* pos_s = reinterpret_cast<int*>(smem + P::off_pos);                // [buf][page|slot][ENC_TILE]
    double* mean_s = reinterpret_cast<double*>(smem + P::off_mean);
    float* rho_s = reinterpret_cast<float*>(smem + P::off_rho);            // [buf][2][ENC_TILE]

    const int kvh = blockIdx.y, side = blockIdx.z;
    const __nv_bfloat16* x_new = side == 0 ? k_new : v_new;
    const double* R = (side == 0 ? rk_d : rv_d) + (size_t)kvh * D * D;      // fragment order [d/4][d][4]
    const double* mean = (side == 0 ? k_mean_d : v_mean_d) + (size_t)kvh * D;
    const float4* cb_g = reinterpret_cast<const float4*>((side == 0 ? cb_k : cb_v) + (size_t)kvh * L * NOVAKV_C * NOVAKV_G);

    const int n_tiles = (n_tokens + ENC_TILE - 1) / ENC_TILE;
    const int tiles_per_cta = blockIdx.z == 0 ? tiles_per_cta_k : tiles_per_cta_v;     // (the two sides may be cut differently)
    const int tile0 = blockIdx.x * tiles_per_cta;
    const int n_local = max(0, min(n_tiles, tile0 + tiles_per_cta) - tile0);
    {
        // a CTA whose token entries are all unused (sequence -1) has nothing to do
        int any = 0;
        const int t_end = min(n_tokens, (tile0 + n_local) * ENC_TILE);
        for (int t = tile0 * ENC_TILE + threadIdx.x; t < t_end; t += ENC_THREADS) any |= tok_seq[t] != -1;
        if (!__syncthreads_or(any)) return;
    }

    // codebook of this (head, side) -> shared memory, once per CTA
    if (!(VSQ && side == 1)) fill_codebook_pairs(reinterpret_cast<float*>(cb_s), cb_g, L);
    for (int i = threadIdx.x; i < D; i += ENC_THREADS) mean_s[i] = mean[i];
    __syncthreads();
    const bool is_transform = threadIdx.x < NT;
    const int tid = is_transform ? threadIdx.x : threadIdx.x - NT;

    if (is_transform) {
        // ---------------- transform warps: fill r_s[buf] and the destinations of tile i ----------------
        // r[t][c] = sum_i xc[t][i] R[i][c] in binary64 on the tensor cores (mma.sync m8n8k4, f64): exact
        // products, binary64 accumulation in blocks of 4 input dimensions taken in index order, one rounding
        // to binary32 at the end.  Warp w owns the 16 columns 16w .. 16w+15 of all 64 tokens: 8 x 2 fragments
        // of 8 tokens x 8 columns, 2 accumulator registers each.  The input dimension is walked in slabs of
        // KS rows: a slab is KS rows of R in fragment order (one contiguous block, asynchronous copy) and the
        // centred inputs xc[64][KS]; slabs are double buffered and slab s + 1 is fetched while slab s is
        // consumed, one barrier of the transform warps per slab.
        constexpr int KS = P::KS, NSLAB = D / KS;
        constexpr int NWT = NT / 32;                    // transform warps
        constexpr int NTILE_N = D / 8 / NWT;            // column fragments per warp: 2 (D=128) or 1 (D=64)
        constexpr int NTILE_M = ENC_TILE / 8;           // token fragments: 8
        static_assert(NSLAB % 2 == 0 && ENC_TILE * KS / 2 == NT && NTILE_N >= 1, "slab mapping");
        const int wt = tid >> 5, lane = tid & 31, fr = lane >> 2, fk = lane & 3;
        const int xt = tid / (KS / 2), xk = (tid % (KS / 2)) * 2;      // this thread's two inputs of a slab
        uint32_t xraw = 0u;
        auto slab_issue = [&](int tile_t0, int tile_valid, int sl) {
            unsigned char* buf_b = smem + P::off_slab + (sl & 1) * P::slab_bytes;
            const uint32_t dst = (uint32_t)__cvta_generic_to_shared(buf_b + P::slab_x_bytes);
            const char* src = reinterpret_cast<const char*>(R + (size_t)sl * KS * D);
#pragma unroll
            for (int q = 0; q < (int)(P::slab_r_bytes / 16 / NT); ++q)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (tid + q * NT) * 16),
                             "l"(src + (size_t)(tid + q * NT) * 16) : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
            xraw = 0u;
            if (xt < tile_valid)
                xraw = *reinterpret_cast<const uint32_t*>(x_new + ((size_t)(tile_t0 + xt) * n_kv_heads + kvh) * D + sl * KS + xk);
        };
        if (n_local > 0) slab_issue(tile0 * ENC_TILE, min(ENC_TILE, n_tokens - tile0 * ENC_TILE), 0);
        for (int i = 0; i < n_local; ++i) {
            const int buf = i & 1;
            const int t0 = (tile0 + i) * ENC_TILE;
            const int n_valid = min(ENC_TILE, n_tokens - t0);
            float* r_s = reinterpret_cast<float*>(smem + P::off_r + buf * P::r_bytes);
            // destination of each token (validated once); written to shared memory when the buffer is free
            int page = -1, slot = 0;
            if (tid < n_valid) {
                const int sq = tok_seq[t0 + tid], pos = tok_pos[t0 + tid];
                if (sq == -1) {
                    // unused entry of the token list: skipped
                } else if (sq < 0 || sq >= n_seq || pos < 0 || pos / NOVAKV_PAGE_TOKENS >= max_pages_per_seq) {
                    atomicOr(dev_status, NOVAKV_DEV_BAD_TOKEN);
                } else {
                    page = page_table[(size_t)sq * max_pages_per_seq + pos / NOVAKV_PAGE_TOKENS];
                    slot = pos % NOVAKV_PAGE_TOKENS;
                    if (page < 0 || page >= n_pages) {
                        atomicOr(dev_status, NOVAKV_DEV_BAD_PAGE);
                        page = -1;
                    } else if (kvh == 0 && side == 0) {
                        atomicMax(&seq_lens[sq], pos + 1);
                    }
                }
            }
            double acc[NTILE_M][NTILE_N][2];
#pragma unroll
            for (int mt = 0; mt < NTILE_M; ++mt)
#pragma unroll
                for (int nt = 0; nt < NTILE_N; ++nt) { acc[mt][nt][0] = 0.0; acc[mt][nt][1] = 0.0; }
#pragma unroll 1
            for (int sl = 0; sl < NSLAB; ++sl) {
                unsigned char* buf_b = smem + P::off_slab + (sl & 1) * P::slab_bytes;
                double* xs = reinterpret_cast<double*>(buf_b);
                const double* Rs = reinterpret_cast<const double*>(buf_b + P::slab_x_bytes);
                // slab sl: its rows of R have landed, its inputs are centred in binary64 (exact) and stored
                asm volatile("cp.async.wait_group 0;" ::: "memory");
                {
                    const __nv_bfloat162 xb = *reinterpret_cast<const __nv_bfloat162*>(&xraw);
                    const bool valid = xt < n_valid;
                    double2 v;
                    v.x = valid ? (double)__bfloat162float(xb.x) - mean_s[sl * KS + xk] : 0.0;
                    v.y = valid ? (double)__bfloat162float(xb.y) - mean_s[sl * KS + xk + 1] : 0.0;
                    *reinterpret_cast<double2*>(xs + ((size_t)(xk >> 2) * ENC_TILE + xt) * 4 + (xk & 3)) = v;   // [k/4][t][k%4]
                }
                nbar_sync(BAR_T, NT);       // slab sl visible; everyone is done with slab sl - 1 (the other buffer)
                if (sl + 1 < NSLAB) slab_issue(t0, n_valid, sl + 1);
                else if (i + 1 < n_local) slab_issue(t0 + ENC_TILE, min(ENC_TILE, n_tokens - t0 - ENC_TILE), 0);
#pragma unroll
                for (int kq = 0; kq < KS / 4; ++kq) {
                    // B fragments: R[4 kq + fk][column 16 wt + 8 nt + fr]; A fragments: xc[token 8 mt + fr][4 kq + fk]
                    double bf[NTILE_N];
#pragma unroll
                    for (int nt = 0; nt < NTILE_N; ++nt) bf[nt] = Rs[((size_t)kq * D + (wt * NTILE_N + nt) * 8 + fr) * 4 + fk];
#pragma unroll
                    for (int mt = 0; mt < NTILE_M; ++mt) {
                        const double af = xs[((size_t)kq * ENC_TILE + mt * 8 + fr) * 4 + fk];
#pragma unroll
                        for (int nt = 0; nt < NTILE_N; ++nt)
                            asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                                         : "+d"(acc[mt][nt][0]), "+d"(acc[mt][nt][1]) : "d"(af), "d"(bf[nt]));
                    }
                }
            }
            if (i >= 2) nbar_sync(BAR_EMPTY + buf, ENC_THREADS);          // the search of tile i-2 has released the buffer
            if (tid < ENC_TILE) {
                pos_s[(buf * 2 + 0) * ENC_TILE + tid] = page;
                pos_s[(buf * 2 + 1) * ENC_TILE + tid] = slot;
            }
            // accumulator fragment: token 8 mt + fr, columns 16 wt + 8 nt + 2 fk, + 1
#pragma unroll
            for (int mt = 0; mt < NTILE_M; ++mt)
#pragma unroll
                for (int nt = 0; nt < NTILE_N; ++nt)
                    *reinterpret_cast<float2*>(r_s + (size_t)(mt * 8 + fr) * RS + (wt * NTILE_N + nt) * 8 + 2 * fk) =
                        make_float2((float)acc[mt][nt][0], (float)acc[mt][nt][1]);
            if (KSC && side == 0) {
                // 4 threads per token, thread `part` takes the columns = part (mod 4): conflict-free rows
                nbar_sync(BAR_T, NT);
                const int t = tid >> 2, part = tid & 3;
                float* row = r_s + (size_t)t * RS + part;
                double ss = 0.0;
#pragma unroll 8
                for (int i = 0; i < D / 4; ++i) {
                    const double r = (double)row[4 * i];
                    ss = fma(r, r, ss);
                }
                ss += __shfl_xor_sync(0xffffffffu, ss, 1);
                ss += __shfl_xor_sync(0xffffffffu, ss, 2);
                float rho = __bfloat162float(__float2bfloat16_rn((float)sqrt(ss / (double)D)));
                if (!(rho > 0.f) || !isfinite(rho)) rho = 1.f;
#pragma unroll 8
                for (int i = 0; i < D / 4; ++i) row[4 * i] = __fdiv_rn(row[4 * i], rho);
                if (part == 0) rho_s[(buf * 2) * ENC_TILE + t] = rho;
            }
            if (VSQ && side == 1) {
                nbar_sync(BAR_T, NT);
                const int t = tid >> 2, part = tid & 3;
                float* row = r_s + (size_t)t * RS + part;
                float mn = row[0], mx = row[0];
#pragma unroll 8
                for (int i = 1; i < D / 4; ++i) { mn = fminf(mn, row[4 * i]); mx = fmaxf(mx, row[4 * i]); }
                mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 1)); mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, 2)); mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float zero = __bfloat162float(__float2bfloat16_rn(mn));
                float scale = __bfloat162float(__float2bfloat16_rn(__fdiv_rn(__fsub_rn(mx, zero), 3.0f)));
                if (!(scale > 0.f) || !isfinite(scale)) scale = 1.f;
#pragma unroll 8
                for (int i = 0; i < D / 4; ++i) {
                    float u = rintf(__fdiv_rn(__fsub_rn(row[4 * i], zero), scale));
                    if (!(u > 0.f)) u = 0.f;
                    row[4 * i] = fminf(u, 3.f);
                }
                if (part == 0) { rho_s[(buf * 2) * ENC_TILE + t] = scale; rho_s[(buf * 2 + 1) * ENC_TILE + t] = zero; }
            }
            __threadfence_block();
            nbar_arrive(BAR_FULL + buf, ENC_THREADS);            // hand tile i to the search warps
        }
    } else {
        // ---------------- search warps: nearest codewords of tile i, paged store ------------------------
        for (int i = 0; i < n_local; ++i) {
            const int buf = i & 1;
            const int t0 = (tile0 + i) * ENC_TILE;
            const int n_valid = min(ENC_TILE, n_tokens - t0);
            const float* r_s = reinterpret_cast<const float*>(smem + P::off_r + buf * P::r_bytes);
            nbar_sync(BAR_FULL + buf, ENC_THREADS);
            if (VSQ && side == 1) {
                // four levels (0..3, held as floats) per byte: the byte of group l
                for (int e = tid; e < ENC_TILE * L; e += NT) {
                    const int t = e / L, l = e - t * L;
                    const float4 c = *reinterpret_cast<const float4*>(r_s + (size_t)t * RS + l * 4);
                    idx_s[e] = (uint8_t)((int)c.x | ((int)c.y << 2) | ((int)c.z << 4) | ((int)c.w << 6));
                }
            } else {
                const __nv_bfloat16* x_tile = x_new + ((size_t)t0 * n_kv_heads + kvh) * D;
                const double* R_plain = (side == 0 ? rk_plain : rv_plain) + (size_t)kvh * D * D;
                // normalised keys are defined in binary32: the values in r_s are the vector to encode
                if (KSC && side == 0)
                    search_tile<D, true>(r_s, cb_s, idx_s, n_valid, tid >> 5, NT / 32, x_tile, (size_t)n_kv_heads * D, mean_s, R_plain);
                else
                    search_tile<D, false>(r_s, cb_s, idx_s, n_valid, tid >> 5, NT / 32, x_tile, (size_t)n_kv_heads * D, mean_s, R_plain);
            }
            nbar_sync(BAR_S, NT);
            for (int e = tid; e < n_valid * L; e += NT) {
                const int t = e / L, l = e - t * L;
                const int page = pos_s[(buf * 2 + 0) * ENC_TILE + t];
                if (page < 0) continue;
                const int slot = pos_s[(buf * 2 + 1) * ENC_TILE + t];
                const size_t base = ((size_t)page * n_kv_heads + kvh) * (NOVAKV_PAGE_TOKENS * L);
                if (side == 0) k_pages[base + novakv_k_offset<L>(slot, l)] = idx_s[e];
                else v_pages[base + novakv_v_offset<L>(slot, l)] = idx_s[e];
            }
            if (KSC && side == 0 && tid < n_valid) {
                const int page = pos_s[(buf * 2 + 0) * ENC_TILE + tid];
                if (page >= 0)
                    k_scales[((size_t)page * n_kv_heads + kvh) * NOVAKV_PAGE_TOKENS + pos_s[(buf * 2 + 1) * ENC_TILE + tid]] =
                        __float2bfloat16_rn(rho_s[(buf * 2) * ENC_TILE + tid]);
            }
            if (VSQ && side == 1 && tid < n_valid) {
                const int page = pos_s[(buf * 2 + 0) * ENC_TILE + tid];
                if (page >= 0)
                    reinterpret_cast<__nv_bfloat162*>(v_meta)[((size_t)page * n_kv_heads + kvh) * NOVAKV_PAGE_TOKENS +
                                                              pos_s[(buf * 2 + 1) * ENC_TILE + tid]] =
                        __floats2bfloat162_rn(rho_s[(buf * 2) * ENC_TILE + tid], rho_s[(buf * 2 + 1) * ENC_TILE + tid]);
            }
            nbar_sync(BAR_S, NT);                                // idx_s and the buffer are free again
            if (i + 2 < n_local) nbar_arrive(BAR_EMPTY + buf, ENC_THREADS);
        }
    }
}

// Append-sized batches (a decode step appends one token per sequence): the tiled kernel above would
// pad every (head, side) to a 64-token tile and fill a 128 KB codebook per CTA.  Here one warp owns one
// group of one (head, side) and stages only its 4 columns of the transform (4 KB of binary64) and its
// group's codebook (4 KB), so the work spreads over L/4 * Hkv * 2 CTAs.  A pass covers tp tokens
// (tp = 1, 2, ... 32, the smallest power of two that holds the batch, at most 32): lane = grp * tp + token.
// The 32 / tp lane groups of a token share its transform (each takes one block of the input dimension, at most 8
// blocks; a butterfly adds the partial sums, so every lane holds the same coefficients) and search disjoint
// ranges of the codebook; their minima are merged with the lowest index winning ties.
// Everything that depends only on the calibration is staged before the grid-dependency wait, so it
// overlaps the tail of the preceding kernel in the stream.
// The coefficients are accumulated in binary64 (index order inside a block, then the blocks pairwise).  The
// search is the certified one of the tiled kernel: binary32 ranking, and a binary64 search by the whole warp
// wherever the two nearest codewords are closer than binary32 rounding can resolve (the binary64 pipe is the
// slowest unit of the SM: a binary64 search of every token was 60 % of this kernel's time after the launch).
// KSC (key format with a per-token scale): the L/4 CTAs of a (head, side) form a thread-block cluster;
// each publishes the sums of squares of its 16 coefficients per token in its shared memory, a cluster
// barrier makes them visible, and every CTA adds the L/4 x 4 partial sums in the same fixed order through
// distributed shared memory, so that all of them normalise by the same rho.
// Binary64 search of one coefficient vector (the same in every lane) against a group's 256 codewords by the
// whole warp: lane i takes codewords i, i + 32, ... in ascending order with a strict '<'; the lanes' minima are
// merged with the lowest index winning ties.  The distance is the plain sum of the four squares, every
// operation rounded to binary64.
__device__ __forceinline__ int exact_search_warp(const double (&rd)[4], const float4* cb /* shared, [256] */, int lane) {
    double best = CUDART_INF;
    int bi = lane;
#pragma unroll
    for (int j = 0; j < NOVAKV_C / 32; ++j) {
        const float4 c = cb[lane + 32 * j];
        const double e0 = rd[0] - (double)c.x, e1 = rd[1] - (double)c.y, e2 = rd[2] - (double)c.z, e3 = rd[3] - (double)c.w;
        const double dd = __dadd_rn(__dadd_rn(__dadd_rn(__dmul_rn(e0, e0), __dmul_rn(e1, e1)), __dmul_rn(e2, e2)), __dmul_rn(e3, e3));
        if (dd < best) { best = dd; bi = lane + 32 * j; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const double ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ob < best || (ob == best && oi < bi)) { best = ob; bi = oi; }
    }
    return bi;
}

template <int D, int FMT>
__global__ void __launch_bounds__(128)
novakv_encode_small_kernel(const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new,
                           const int32_t* __restrict__ tok_seq, const int32_t* __restrict__ tok_pos, int n_tokens,
                           int tp_log2,
                           const double* __restrict__ rk_d, const double* __restrict__ rv_d,
                           const double* __restrict__ k_mean_d, const double* __restrict__ v_mean_d,
                           const float* __restrict__ cb_k, const float* __restrict__ cb_v,
                           uint8_t* __restrict__ k_pages, uint8_t* __restrict__ v_pages,
                           __nv_bfloat16* __restrict__ k_scales, __nv_bfloat16* __restrict__ v_meta, int n_pages,
                           const int32_t* __restrict__ page_table, int max_pages_per_seq, int n_seq,
                           int32_t* __restrict__ seq_lens, int n_kv_heads, uint32_t* __restrict__ dev_status) {
    constexpr int L = D / NOVAKV_G;
    constexpr bool KSC = FMT >= 1, VSQ = FMT == 2;
    // Rows of the transform and the mean are indexed by i + i / (D / 4): one row of padding after every quarter of
    // the input dimension, so that lane groups working on different blocks of it read different banks.
    constexpr int DP = D + 4;
    auto padded = [](int i) { return i + i / (D / 4); };
    __shared__ __align__(16) double R_s[4][DP][4];
    __shared__ float4 cb_s[4][NOVAKV_C];
    __shared__ double mean_s[DP];
    __shared__ double ss_s[4][32];                  // KSC: sum of squares of a warp's 4 coefficients, per token of the pass
    __shared__ float mx_s[4][32];                   // VSQ: maximum of a warp's 4 value coefficients (the minimum rides in ss_s)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int l = blockIdx.x * 4 + warp, kvh = blockIdx.y, side = blockIdx.z;
    const __nv_bfloat16* x_new = side == 0 ? k_new : v_new;
    const double* R = (side == 0 ? rk_d : rv_d) + (size_t)kvh * D * D;
    const double* mean = (side == 0 ? k_mean_d : v_mean_d) + (size_t)kvh * D;
    const float4* cb_g = reinterpret_cast<const float4*>((side == 0 ? cb_k : cb_v) + ((size_t)kvh * L + l) * NOVAKV_C * NOVAKV_G);
#ifdef NOVAKV_TIMING
    long long tm[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
    long long t_prev = clock64();
    unsigned long long g_a0, g_a1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g_a0));
#define NOVAKV_ETICK(i) { const long long t_now = clock64(); tm[i] += t_now - t_prev; t_prev = t_now; }
#else
#define NOVAKV_ETICK(i)
#endif
    {
        // calibration constants -> shared memory; every load is issued before the first store
        double2 ra[D / 32], rb[D / 32];
        float4 cw[NOVAKV_C / 32];
#pragma unroll
        for (int k = 0; k < D / 32; ++k) {
            ra[k] = *reinterpret_cast<const double2*>(R + (size_t)(lane + 32 * k) * D + l * 4);
            rb[k] = *reinterpret_cast<const double2*>(R + (size_t)(lane + 32 * k) * D + l * 4 + 2);
        }
#pragma unroll
        for (int k = 0; k < NOVAKV_C / 32; ++k) cw[k] = cb_g[lane + 32 * k];
        const double mv = threadIdx.x < D ? mean[threadIdx.x] : 0.0;
#pragma unroll
        for (int k = 0; k < D / 32; ++k) {
            *reinterpret_cast<double2*>(&R_s[warp][padded(lane + 32 * k)][0]) = ra[k];
            *reinterpret_cast<double2*>(&R_s[warp][padded(lane + 32 * k)][2]) = rb[k];
        }
#pragma unroll
        for (int k = 0; k < NOVAKV_C / 32; ++k) cb_s[warp][lane + 32 * k] = cw[k];
        if (threadIdx.x < D) mean_s[padded(threadIdx.x)] = mv;
    }
    __syncthreads();
    NOVAKV_ETICK(0)
    novakv_grid_dependency_wait();           // inputs and the cache may be written by preceding kernels
    NOVAKV_ETICK(1)

    const int tp = 1 << tp_log2;
    const int tok_in_pass = lane & (tp - 1), grp = lane >> tp_log2;
    const int codes_per_grp = NOVAKV_C >> (5 - tp_log2);
    const int c0 = grp * codes_per_grp;
    const bool reporter = blockIdx.x == 0 && warp == 0 && kvh == 0 && side == 0 && grp == 0;
    // the lane groups of a token also share its transform: each takes one block of the input dimension
    // (at most 8 blocks), and a butterfly over the lane groups adds the partial sums
    const int ts_log2 = min(5 - tp_log2, 3);
    const int part = grp & ((1 << ts_log2) - 1);
    const int per = (D / 8) >> ts_log2;             // 16-byte chunks of the token row per lane (>= 1)

    for (int t0 = 0; t0 < n_tokens; t0 += tp) {
        const int tkn = t0 + tok_in_pass;
        const bool in_range = tkn < n_tokens;
        int s = -1, pos = 0;
        if (in_range) { s = tok_seq[tkn]; pos = tok_pos[tkn]; }
        // this lane's block of its token's row (the loads are in flight together with the token list's)
        uint4 xr[D / 8];
        const uint4* xrow = reinterpret_cast<const uint4*>(x_new + ((size_t)(in_range ? tkn : 0) * n_kv_heads + kvh) * D) + part * per;
#pragma unroll
        for (int c = 0; c < D / 8; ++c)
            if (c < per) xr[c] = xrow[c];
        // a pass whose entries are all unused does nothing (the same decision in every warp and CTA: it depends
        // on the token list alone)
        if (!__any_sync(0xffffffffu, s != -1)) continue;
        // destination: the page-table entry is requested here and looked at after the transform
        const bool ok = s >= 0 && s < n_seq && pos >= 0 && pos / NOVAKV_PAGE_TOKENS < max_pages_per_seq;
        if (s != -1 && !ok && reporter) atomicOr(dev_status, NOVAKV_DEV_BAD_TOKEN);
        int page_raw = -1;
        if (ok) page_raw = page_table[(size_t)s * max_pages_per_seq + pos / NOVAKV_PAGE_TOKENS];
        const int slot = pos % NOVAKV_PAGE_TOKENS;
        NOVAKV_ETICK(2)
        // coefficients of group l in binary64: every block of the input dimension in index order, then the blocks
        // pairwise (neighbours first); all lanes of a token end with the same bits
        double acc0 = 0.0, acc1 = 0.0, acc2 = 0.0, acc3 = 0.0;
#pragma unroll
        for (int c = 0; c < D / 8; ++c) {
            if (c < per) {
                const __nv_bfloat16* xb = reinterpret_cast<const __nv_bfloat16*>(&xr[c]);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int i = padded((part * per + c) * 8 + j);
                    const double xc = (double)__bfloat162float(xb[j]) - mean_s[i];
                    const double2 r01 = *reinterpret_cast<const double2*>(&R_s[warp][i][0]);
                    const double2 r23 = *reinterpret_cast<const double2*>(&R_s[warp][i][2]);
                    acc0 = fma(xc, r01.x, acc0);
                    acc1 = fma(xc, r01.y, acc1);
                    acc2 = fma(xc, r23.x, acc2);
                    acc3 = fma(xc, r23.y, acc3);
                }
            }
        }
        for (int b = 0; b < ts_log2; ++b) {
            const int off = tp << b;
            acc0 += __shfl_xor_sync(0xffffffffu, acc0, off);
            acc1 += __shfl_xor_sync(0xffffffffu, acc1, off);
            acc2 += __shfl_xor_sync(0xffffffffu, acc2, off);
            acc3 += __shfl_xor_sync(0xffffffffu, acc3, off);
        }
        int page = -1;
        if (ok) {
            if (page_raw < 0 || page_raw >= n_pages) {
                if (reporter) atomicOr(dev_status, NOVAKV_DEV_BAD_PAGE);
            } else {
                page = page_raw;
                if (reporter) atomicMax(&seq_lens[s], pos + 1);
            }
        }
        float4 r = make_float4((float)acc0, (float)acc1, (float)acc2, (float)acc3);
        NOVAKV_ETICK(3)
        int vsq_byte = 0;
        if (KSC) {
            namespace cg = cooperative_groups;
            cg::cluster_group cluster = cg::this_cluster();
            if (side == 0 && grp == 0) {
                double ss = (double)r.x * (double)r.x;
                ss = fma((double)r.y, (double)r.y, ss);
                ss = fma((double)r.z, (double)r.z, ss);
                ss = fma((double)r.w, (double)r.w, ss);
                ss_s[warp][tok_in_pass] = ss;
            }
            cluster.sync();                             // every CTA of the (head, side) has published its partial sums
            if (side == 0) {
                double tot = 0.0;
                for (unsigned cr = 0; cr < cluster.num_blocks(); ++cr) {
                    const double* remote = cluster.map_shared_rank(&ss_s[0][0], cr);
#pragma unroll
                    for (int w = 0; w < 4; ++w) tot += remote[w * 32 + tok_in_pass];
                }
                float rho = __bfloat162float(__float2bfloat16_rn((float)sqrt(tot / (double)D)));
                if (!(rho > 0.f) || !isfinite(rho)) rho = 1.f;
                r = make_float4(__fdiv_rn(r.x, rho), __fdiv_rn(r.y, rho), __fdiv_rn(r.z, rho), __fdiv_rn(r.w, rho));
                if (blockIdx.x == 0 && warp == 0 && grp == 0 && page >= 0)
                    k_scales[((size_t)page * n_kv_heads + kvh) * NOVAKV_PAGE_TOKENS + slot] = __float2bfloat16_rn(rho);
            }
            if (VSQ && side == 1 && grp == 0) {
                // value side: the warp's minimum and maximum travel in the same slots (as doubles)
                ss_s[warp][tok_in_pass] = (double)fminf(fminf(r.x, r.y), fminf(r.z, r.w));
                mx_s[warp][tok_in_pass] = fmaxf(fmaxf(r.x, r.y), fmaxf(r.z, r.w));
            }
            if (VSQ) cluster.sync();
            if (VSQ && side == 1) {
                float mn = CUDART_INF_F, mx = -CUDART_INF_F;
                for (unsigned cr = 0; cr < cluster.num_blocks(); ++cr) {
                    const double* rmn = cluster.map_shared_rank(&ss_s[0][0], cr);
                    const float* rmx = cluster.map_shared_rank(&mx_s[0][0], cr);
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        mn = fminf(mn, (float)rmn[w * 32 + tok_in_pass]);
                        mx = fmaxf(mx, rmx[w * 32 + tok_in_pass]);
                    }
                }
                const float zero = __bfloat162float(__float2bfloat16_rn(mn));
                float scale = __bfloat162float(__float2bfloat16_rn(__fdiv_rn(__fsub_rn(mx, zero), 3.0f)));
                if (!(scale > 0.f) || !isfinite(scale)) scale = 1.f;
                auto level = [&](float x) {
                    float u = rintf(__fdiv_rn(__fsub_rn(x, zero), scale));
                    if (!(u > 0.f)) u = 0.f;
                    return (int)fminf(u, 3.f);
                };
                vsq_byte = level(r.x) | (level(r.y) << 2) | (level(r.z) << 4) | (level(r.w) << 6);
                if (blockIdx.x == 0 && warp == 0 && grp == 0 && page >= 0)
                    reinterpret_cast<__nv_bfloat162*>(v_meta)[((size_t)page * n_kv_heads + kvh) * NOVAKV_PAGE_TOKENS + slot] =
                        __floats2bfloat162_rn(scale, zero);
            }
            cluster.sync();                             // partial sums may be overwritten by the next pass / CTAs may exit
        }
        // The vector to encode is the binary64 coefficient; for normalised keys it is the binary32 quotient.
        double rd[4] = {acc0, acc1, acc2, acc3};
        if (KSC && side == 0) { rd[0] = (double)r.x; rd[1] = (double)r.y; rd[2] = (double)r.z; rd[3] = (double)r.w; }
        // Certified search, as in the tiled kernel: this lane group's range of the codebook is ranked in binary32
        // from the coefficient rounded to binary32 (first minimum in ascending order), with the second-smallest
        // distance tracked beside the smallest (equal distances count as two: their gap is zero).
        // The range is a whole number of blocks of 8 codewords.  Per block the 8 distances are independent; the block
        // minimum updates the running minimum with a strict '<' (keeps the first block that attains it), and the
        // larger of the two feeds the second-smallest value.  The winning block is then evaluated again (same
        // instructions, same bits): its first distance equal to the minimum gives the index, the others are the
        // remaining candidates for the second-smallest value.
        const float4* cbw = &cb_s[warp][c0];
        auto dist8 = [&](int blk, float (&d)[8]) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const float4 cw = cbw[blk * 8 + k];
                const float e0 = r.x - cw.x, e1 = r.y - cw.y, e2 = r.z - cw.z, e3 = r.w - cw.w;
                d[k] = fmaf(e3, e3, fmaf(e2, e2, fmaf(e1, e1, e0 * e0)));
            }
        };
        float best = CUDART_INF_F, sec = CUDART_INF_F;
        int bblk = 0;
#pragma unroll 2
        for (int blk = 0; blk < codes_per_grp / 8; ++blk) {
            float d[8];
            dist8(blk, d);
            const float m = fminf(fminf(fminf(d[0], d[1]), fminf(d[2], d[3])), fminf(fminf(d[4], d[5]), fminf(d[6], d[7])));
            sec = fminf(sec, fmaxf(best, m));
            if (m < best) { best = m; bblk = blk; }
        }
        int bi;
        {
            float d[8];
            dist8(bblk, d);
            int kb = 7;
#pragma unroll
            for (int k = 6; k >= 0; --k)
                if (d[k] == best) kb = k;
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (k != kb) sec = fminf(sec, d[k]);
            bi = c0 + bblk * 8 + kb;
        }
        NOVAKV_ETICK(6)
        // merge the groups of a token: smaller distance wins, equal distances keep the lower index
        for (int off = tp; off < 32; off <<= 1) {
            const float ob = __shfl_xor_sync(0xffffffffu, best, off);
            const float os = __shfl_xor_sync(0xffffffffu, sec, off);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
            sec = fminf(fminf(sec, os), fmaxf(best, ob));
            if (ob < best || (ob == best && oi < bi)) { best = ob; bi = oi; }
        }
        NOVAKV_ETICK(7)
        // Where binary32 rounding (of the coefficient: at most 2^-24 per component, none for the quotient, which is
        // a binary32 number; and of the distance) can have changed the order of the two nearest codewords, the whole
        // warp searches that token's group again in binary64.
        {
            float delta = 0.f;
            if (!(KSC && side == 0))
                delta = 5.97e-8f * sqrtf(fmaf(r.x, r.x, fmaf(r.y, r.y, fmaf(r.z, r.z, r.w * r.w)))) * 1.0001f;
            const bool need = grp == 0 && s != -1 && !(VSQ && side == 1) && needs_exact_search(best, sec, delta);
            unsigned todo = __ballot_sync(0xffffffffu, need);
#ifdef NOVAKV_TIMING
            tm[8] += __popc(todo);
#endif
            while (todo) {
                const int src = __ffs(todo) - 1;             // (a lane of lane group 0: its index is the token's)
                todo &= todo - 1;
                const double rs[4] = {__shfl_sync(0xffffffffu, rd[0], src), __shfl_sync(0xffffffffu, rd[1], src),
                                      __shfl_sync(0xffffffffu, rd[2], src), __shfl_sync(0xffffffffu, rd[3], src)};
                const int res = exact_search_warp(rs, cb_s[warp], lane);
                if (tok_in_pass == src) bi = res;
            }
        }
        NOVAKV_ETICK(4)
        if (VSQ && side == 1) bi = vsq_byte;             // scalar codec: the byte holds four levels, no search result
        if (grp == 0 && page >= 0) {
            const size_t base = ((size_t)page * n_kv_heads + kvh) * (NOVAKV_PAGE_TOKENS * L);
            if (side == 0) k_pages[base + novakv_k_offset<L>(slot, l)] = (uint8_t)bi;
            else v_pages[base + novakv_v_offset<L>(slot, l)] = (uint8_t)bi;
        }
    }
#ifdef NOVAKV_TIMING
    NOVAKV_ETICK(5)
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(g_a1));
    if (threadIdx.x == 0 && blockIdx.y == 0 && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1))
        printf("append cta (%d,%d,%d) clocks: constants %lld dependency wait %lld rows+lookup %lld transform %lld ranking %lld merge %lld certificate+re-search %lld (%lld re-searches) store %lld | ns start %llu end %llu\n",
               blockIdx.x, blockIdx.y, blockIdx.z, tm[0], tm[1], tm[2], tm[3], tm[6], tm[7], tm[4], tm[8], tm[5], g_a0, g_a1);
#endif
}

// Search only, from given binary32 coefficients [n][Hkv][D]; logical indices out [n][Hkv][L].
template <int D>
__global__ void __launch_bounds__(ENC_THREADS, 1)
novakv_search_kernel(const float* __restrict__ coef, int n, const float* __restrict__ cb_all, int n_kv_heads,
                     uint8_t* __restrict__ idx_out) {
    constexpr int L = D / NOVAKV_G;
    constexpr int RS = EncSmem<D>::RSTRIDE;
    extern __shared__ __align__(16) unsigned char smem[];
    float4* cb_s = reinterpret_cast<float4*>(smem);
    float* r_s = reinterpret_cast<float*>(smem + EncSmem<D>::cb_bytes);
    uint8_t* idx_s = smem + EncSmem<D>::cb_bytes + EncSmem<D>::r_bytes;
    const int kvh = blockIdx.y;
    const float4* cb_g = reinterpret_cast<const float4*>(cb_all + (size_t)kvh * L * NOVAKV_C * NOVAKV_G);
    fill_codebook_pairs(reinterpret_cast<float*>(cb_s), cb_g, L);
    const int n_tiles = (n + ENC_TILE - 1) / ENC_TILE;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const int t0 = tile * ENC_TILE;
        const int n_valid = min(ENC_TILE, n - t0);
        __syncthreads();
        for (int i = threadIdx.x; i < ENC_TILE * D; i += ENC_THREADS) {
            const int t = i / D, c = i - t * D;
            r_s[(size_t)t * RS + c] = t < n_valid ? coef[((size_t)(t0 + t) * n_kv_heads + kvh) * D + c] : 0.f;
        }
        __syncthreads();
        search_tile<D, true>(r_s, cb_s, idx_s, n_valid, threadIdx.x >> 5, ENC_THREADS / 32, nullptr, 0, nullptr, nullptr);
        __syncthreads();
        for (int i = threadIdx.x; i < n_valid * L; i += ENC_THREADS) {
            const int t = i / L, l = i - t * L;
            idx_out[((size_t)(t0 + t) * n_kv_heads + kvh) * L + l] = idx_s[i];
        }
    }
}

template <int D>
novakv_status launch_encode_t(novakv_ctx* ctx, const novakv_layer& ly, const __nv_bfloat16* k_new,
                              const __nv_bfloat16* v_new, const int32_t* tok_seq, const int32_t* tok_pos,
                              int n_tokens, uint8_t* k_pages, uint8_t* v_pages, int n_pages,
                              const int32_t* page_table, int max_pages_per_seq, int n_seq, int32_t* seq_lens,
                              cudaStream_t stream, __nv_bfloat16* k_scales, __nv_bfloat16* v_meta) {
    if (n_tokens <= NOVAKV_SMALL_APPEND_TOKENS) {
        dim3 grid(D / NOVAKV_G / 4, ctx->cfg.n_kv_heads, 2);
        novakv_prof_scope ps(ctx, 1, stream);
        int tp_log2 = 0;
        while ((1 << tp_log2) < n_tokens && tp_log2 < 5) ++tp_log2;
        auto small = v_meta ? novakv_encode_small_kernel<D, 2>
                            : (k_scales ? novakv_encode_small_kernel<D, 1> : novakv_encode_small_kernel<D, 0>);
        if (k_scales == nullptr) {
            novakv_launch_pdl(novakv_encode_small_kernel<D, 0>, grid, dim3(128), 0, stream, k_new, v_new, tok_seq, tok_pos,
                              n_tokens, tp_log2, ly.rk_d, ly.rv_d, ly.k_mean_d, ly.v_mean_d, ly.cb_k, ly.cb_v, k_pages, v_pages,
                              (__nv_bfloat16*)nullptr, (__nv_bfloat16*)nullptr, n_pages, page_table, max_pages_per_seq, n_seq, seq_lens,
                              ctx->cfg.n_kv_heads, ctx->dev_status);
        } else {
            // scaled key format: the L/4 CTAs of a (head, side) are one cluster (8 at d = 128, 4 at d = 64)
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = grid;
            cfg.blockDim = dim3(128);
            cfg.stream = stream;
            cudaLaunchAttribute attr[2];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            attr[1].id = cudaLaunchAttributeClusterDimension;
            attr[1].val.clusterDim.x = grid.x;
            attr[1].val.clusterDim.y = 1;
            attr[1].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 2;
            const int hkv = ctx->cfg.n_kv_heads;
            if (cudaLaunchKernelEx(&cfg, small, k_new, v_new, tok_seq, tok_pos, n_tokens, tp_log2,
                                   (const double*)ly.rk_d, (const double*)ly.rv_d, (const double*)ly.k_mean_d,
                                   (const double*)ly.v_mean_d, (const float*)ly.cb_k, (const float*)ly.cb_v, k_pages, v_pages,
                                   k_scales, v_meta, n_pages, page_table, max_pages_per_seq, n_seq, seq_lens, hkv,
                                   ctx->dev_status) != cudaSuccess)
                return NOVAKV_ECUDA;
        }
        ps.end();
        ctx->launches++;
        return cudaGetLastError() == cudaSuccess ? NOVAKV_OK : NOVAKV_ECUDA;
    }
    auto kern = v_meta ? novakv_encode_kernel<D, 2> : (k_scales ? novakv_encode_kernel<D, 1> : novakv_encode_kernel<D, 0>);
    const size_t smem = EncPipe<D>::total;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return NOVAKV_ECUDA;
    const int n_tiles = (n_tokens + ENC_TILE - 1) / ENC_TILE;
    const int hs = ctx->cfg.n_kv_heads * 2;
    // enough CTAs per (head, side) to fill the machine about twice, each amortising its codebook fill
    // CTAs per (head, side): whole waves of the machine, each CTA amortising its 128 KB codebook fill
    // (counted as 1.5 tiles) over several tiles
    int ctas_x = 1, tiles_per_cta = n_tiles;
    double best = 1e30;
    for (int w = 1; w <= 8; ++w) {
        int cx = min(n_tiles, max(1, (w * ctx->n_sm) / hs));
        const int tp = (n_tiles + cx - 1) / cx;
        cx = (n_tiles + tp - 1) / tp;
        const int waves = (cx * hs + ctx->n_sm - 1) / ctx->n_sm;
        const double cost = waves * (tp + 1.5);
        if (cost < best) { best = cost; ctas_x = cx; tiles_per_cta = tp; }
    }
    int tiles_k = tiles_per_cta, tiles_v = tiles_per_cta;
    if (v_meta != nullptr && ctas_x > 1) {
        // scalar INT2 values need no codeword search: a value tile costs about 3/8 of a key tile, so the CTAs of a head
        // are shared out 8 : 3 between the two sides instead of evenly (the value side then takes longer runs)
        const int per_head = 2 * ctas_x;
        const int ck = max(1, min(n_tiles, (per_head * 8 + 5) / 11)), cv = max(1, min(n_tiles, per_head - ck));
        tiles_k = (n_tiles + ck - 1) / ck;
        tiles_v = (n_tiles + cv - 1) / cv;
        ctas_x = max((n_tiles + tiles_k - 1) / tiles_k, (n_tiles + tiles_v - 1) / tiles_v);
    }
    dim3 grid(ctas_x, ctx->cfg.n_kv_heads, 2);
    novakv_prof_scope ps(ctx, 1, stream);
    kern<<<grid, ENC_THREADS, smem, stream>>>(k_new, v_new, tok_seq, tok_pos, n_tokens, ly.rk_d_mma, ly.rv_d_mma,
                                               ly.rk_d, ly.rv_d, ly.k_mean_d, ly.v_mean_d, ly.cb_k, ly.cb_v, k_pages, v_pages, k_scales,
                                               v_meta, n_pages, page_table, max_pages_per_seq, n_seq, seq_lens,
                                               ctx->cfg.n_kv_heads, tiles_k, tiles_v, ctx->dev_status);
    ps.end();
    ctx->launches++;
    return cudaGetLastError() == cudaSuccess ? NOVAKV_OK : NOVAKV_ECUDA;
}

template <int D>
novakv_status launch_search_t(novakv_ctx* ctx, const novakv_layer& ly, int which, const float* coef, int n,
                              uint8_t* idx_out, cudaStream_t stream) {
    auto kern = novakv_search_kernel<D>;
    const size_t smem = EncSmem<D>::total;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return NOVAKV_ECUDA;
    const int n_tiles = (n + ENC_TILE - 1) / ENC_TILE;
    // CTAs per head: about two whole waves of the machine
    dim3 grid(max(1, min(n_tiles, (2 * ctx->n_sm) / ctx->cfg.n_kv_heads)), ctx->cfg.n_kv_heads);
    kern<<<grid, ENC_THREADS, smem, stream>>>(coef, n, which == 0 ? ly.cb_k : ly.cb_v, ctx->cfg.n_kv_heads, idx_out);
    ctx->launches++;
    return cudaGetLastError() == cudaSuccess ? NOVAKV_OK : NOVAKV_ECUDA;
}

}  // namespace

novakv_status novakv_launch_encode(novakv_ctx* ctx, const novakv_layer& ly, const __nv_bfloat16* k_new,
    const __nv_bfloat16* v_new, const int32_t* tok_seq, const int32_t* tok_pos, int n_tokens,
    uint8_t* k_pages, uint8_t* v_pages, int n_pages, const int32_t* page_table,
    int max_pages_per_seq, int n_seq, int32_t* seq_lens, cudaStream_t stream, __nv_bfloat16* k_scales,
    __nv_bfloat16* v_meta) {
    if (v_meta != nullptr && k_scales == nullptr) return NOVAKV_EUNSUPPORTED;   // INT2 values come with scaled keys
    if (ctx->cfg.head_dim == 128)
        return launch_encode_t<128>(ctx, ly, k_new, v_new, tok_seq, tok_pos, n_tokens, k_pages, v_pages, n_pages,
                                    page_table, max_pages_per_seq, n_seq, seq_lens, stream, k_scales, v_meta);
    return launch_encode_t<64>(ctx, ly, k_new, v_new, tok_seq, tok_pos, n_tokens, k_pages, v_pages, n_pages,
                               page_table, max_pages_per_seq, n_seq, seq_lens, stream, k_scales, v_meta);
}

// Gather of up to 5 page-locked host buffers into device staging: every 32-bit word crosses the bus
// once, consecutive threads take consecutive words (128-byte requests per warp).
__global__ void __launch_bounds__(256) novakv_stage_kernel(const novakv_stage_args a) {
    // the kernels behind this one in the stream may start their own prologues (calibration constants) now; they
    // wait for this grid's completion before they touch the staged inputs
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const unsigned stride = gridDim.x * blockDim.x;
#pragma unroll 1
    for (int sgm = 0; sgm < a.n; ++sgm) {
        const uint32_t* __restrict__ src = a.src[sgm];
        uint32_t* __restrict__ dst = a.dst[sgm];
        const unsigned words = a.words[sgm];
        if (((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15) == 0 && (words & 3) == 0) {
            // 16 bytes per thread: a quarter of the read requests that cross the bus
            const uint4* __restrict__ s4 = reinterpret_cast<const uint4*>(src);
            uint4* __restrict__ d4 = reinterpret_cast<uint4*>(dst);
            for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < words / 4; i += stride) d4[i] = s4[i];
        } else {
            for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < words; i += stride) dst[i] = src[i];
        }
    }
}

novakv_status novakv_launch_stage(novakv_ctx* ctx, const novakv_stage_args& a, cudaStream_t stream) {
    unsigned total = 0;
    for (int i = 0; i < a.n; ++i) total += a.words[i];
    if (total == 0) return NOVAKV_OK;
    unsigned blocks = (total / 4 + 255) / 256;          // one 16-byte word per thread where the buffers allow it
    if (blocks == 0) blocks = 1;
    if (blocks > (unsigned)(2 * ctx->n_sm)) blocks = 2 * ctx->n_sm;
    novakv_stage_kernel<<<blocks, 256, 0, stream>>>(a);
    ctx->launches++;
    return cudaGetLastError() == cudaSuccess ? NOVAKV_OK : NOVAKV_ECUDA;
}

// ------------------------------------------------------------------------------------------------
// BF16 band, write side: one new token per sequence (App. B "Sink-plus-recent band")
// ------------------------------------------------------------------------------------------------
// One block per sequence.  Thread 0 advances the sequence's (sink_cnt, ring_start, ring_len, quantised
// length); the block copies the new token into its band slot and, when the ring has reached n_rec + block
// tokens, copies the block oldest ring tokens to the staging rows b * block + i with their (sequence,
// position) entries.  Rows of sequences that flush nothing get the "unused" marker (sequence -1).
__global__ void __launch_bounds__(256)
novakv_band_insert_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new, uint4* __restrict__ band_k,
                          uint4* __restrict__ band_v, int band_cap, int n_sink, int n_rec, int block,
                          int32_t* __restrict__ band_meta, int32_t* __restrict__ quant_lens, int row_u4 /* Hkv * d / 8 */,
                          uint4* __restrict__ stage_k, uint4* __restrict__ stage_v, int32_t* __restrict__ tok_seq,
                          int32_t* __restrict__ tok_pos) {
    const int b = blockIdx.x;
    const int ring_cap = band_cap - n_sink;
    __shared__ int s_slot, s_flush, s_rs, s_q;
    if (threadIdx.x == 0) {
        int sc = band_meta[b * 3], rs = band_meta[b * 3 + 1], rl = band_meta[b * 3 + 2], q = quant_lens[b];
        // (state written by this kernel stays in range; a caller's out-of-range state is pulled back into it)
        sc = min(max(sc, 0), n_sink);
        rs = min(max(rs, 0), ring_cap - 1);
        rl = min(max(rl, 0), n_rec + block - 1);
        q = max(q, 0);
        int slot;
        if (sc < n_sink) { slot = sc; ++sc; }
        else { slot = n_sink + (rs + rl) % ring_cap; ++rl; }
        const int flush = rl >= n_rec + block;
        s_slot = slot; s_flush = flush; s_rs = rs; s_q = q;
        if (flush) { rs = (rs + block) % ring_cap; rl -= block; q += block; }
        band_meta[b * 3] = sc; band_meta[b * 3 + 1] = rs; band_meta[b * 3 + 2] = rl;
        quant_lens[b] = q;
    }
    __syncthreads();
    {
        const size_t dst = ((size_t)b * band_cap + s_slot) * row_u4, src = (size_t)b * row_u4;
        for (int i = threadIdx.x; i < row_u4; i += blockDim.x) { band_k[dst + i] = k_new[src + i]; band_v[dst + i] = v_new[src + i]; }
    }
    if (s_flush) {
        // the new token's slot is not among the block oldest ones (the ring holds at least n_rec > 0 more)
        for (int i = threadIdx.x; i < block * row_u4; i += blockDim.x) {
            const int t = i / row_u4, w = i - t * row_u4;
            const size_t src = ((size_t)b * band_cap + n_sink + (s_rs + t) % ring_cap) * row_u4 + w;
            const size_t dst = ((size_t)b * block + t) * row_u4 + w;
            stage_k[dst] = band_k[src];
            stage_v[dst] = band_v[src];
        }
    }
    for (int t = threadIdx.x; t < block; t += blockDim.x) {
        tok_seq[b * block + t] = s_flush ? b : -1;
        tok_pos[b * block + t] = n_sink + s_q + t;
    }
}

novakv_status novakv_launch_band_insert(novakv_ctx* ctx, const void* k_new, const void* v_new, int batch, void* band_k,
    void* band_v, int band_cap, int n_sink, int n_rec, int block, int32_t* band_meta, int32_t* quant_lens,
    void* stage_k, void* stage_v, int32_t* tok_seq, int32_t* tok_pos, cudaStream_t stream) {
    const int row_u4 = ctx->cfg.n_kv_heads * ctx->cfg.head_dim / 8;
    novakv_band_insert_kernel<<<batch, 256, 0, stream>>>((const uint4*)k_new, (const uint4*)v_new, (uint4*)band_k, (uint4*)band_v,
                                                        band_cap, n_sink, n_rec, block, band_meta, quant_lens, row_u4,
                                                        (uint4*)stage_k, (uint4*)stage_v, tok_seq, tok_pos);
    ctx->launches++;
    return cudaGetLastError() == cudaSuccess ? NOVAKV_OK : NOVAKV_ECUDA;
}

novakv_status novakv_launch_search(novakv_ctx* ctx, const novakv_layer& ly, int which, const float* coef,
    int n, uint8_t* idx_out, cudaStream_t stream) {
    if (ctx->cfg.head_dim == 128) return launch_search_t<128>(ctx, ly, which, coef, n, idx_out, stream);
    return launch_search_t<64>(ctx, ly, which, coef, n, idx_out, stream);
}
