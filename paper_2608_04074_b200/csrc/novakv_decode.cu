// Read path: decode-step attention straight from the packed index cache.
//
//   prepare  : q' = sm_scale*log2(e) * q rk_inv_t  per head, and a prefix sum of page counts (the
//              work list of the scan kernel: one unit = one 64-token page of one (sequence, KV head)).
//   stage 1  : persistent scan kernel, one CTA per SM.  Each CTA takes a contiguous range of the
//              global page sequence, so that consecutive pages mostly belong to the same
//              (sequence, KV head) and reuse its score table.  Per (sequence, KV head) segment:
//                - score table LUT[h][l][c] = <q'_h[4l..4l+3], cb_k[l][c]> in shared memory,
//                - a producer warp streams 64-token index chunks into a shared-memory ring with
//                  1-D bulk asynchronous copies (mbarrier completion),
//                - consumer warps: lane <-> token, 32 table lookups summed in registers (no cross
//                  lane reduction), online softmax per 32-token tile, then accumulation of
//                  p * value-codeword in the value-transform domain: a dense [heads x tokens] x
//                  [tokens x d] contraction, run on tensor cores (mma.sync, fp16 operands, fp32
//                  accumulators) or, as the selectable alternative, on CUDA cores in fp32,
//                - the warps' partial (m, l, acc) are merged and written once per segment.
//   merge    : exact log-sum-exp merge of the partials of every (sequence, KV head), then the inverse
//              value transform o = o' rv^T + v_mean, once per head.
//
// Shared-memory gathers are laid out so that a warp's 128-bit table reads never bank-conflict:
// the 8 lanes of a quarter warp always address 8 different 16-byte bank groups ("slots").
#include <math_constants.h>

#include "novakv_internal.cuh"

namespace {

#ifndef NOVAKV_NCW
#define NOVAKV_NCW 8
#endif
// 1: the producer prefetches the pages of its next batch of 32 page ids into L2; 0: no prefetch
#ifndef NOVAKV_L2_PREFETCH_PAGES
#define NOVAKV_L2_PREFETCH_PAGES 0
#endif
#ifndef NOVAKV_PRODUCER_PAGES
#define NOVAKV_PRODUCER_PAGES 4              // pages issued per producer instruction group (2 lanes per page)
#endif
constexpr int NCW = NOVAKV_NCW;               // consumer warps
constexpr int S1_THREADS = (NCW + 1) * 32;    // + one producer warp
constexpr int LUT_PLANE_BYTES = 256 * 256;    // 256 codes x 16 entries x 16 bytes
constexpr int VCB_BYTES = 256 * 256;          // 256 codes x 32 slots x 4 halves
constexpr float M_INIT = -1.0e30f;

// VM selects the value side: false = CUDA cores (fp32 FMA, weights broadcast from shared memory),
// true = tensor cores (mma.sync m16n8k16, fp16 weights and codewords, fp32 accumulators).
template <int D, int HG, bool VM>
struct S1 {
    static constexpr int L = D / NOVAKV_G;
    static constexpr int GPS = L / 8;                         // groups per slot: 4 (d=128) or 2 (d=64)
    static constexpr int PLANES = GPS / 2;
    static constexpr int NGB = L / 8;                         // group blocks of 8 groups (value side, MMA rows)
    static constexpr int HSETS = HG <= 4 ? 1 : 2;             // table entries are 4 heads wide
    static constexpr int HPAD = HSETS * 4;
    static constexpr int CHUNK = NOVAKV_PAGE_TOKENS * L;      // bytes of one page of one head, K or V
    static constexpr int LUT_BYTES = HSETS * PLANES * LUT_PLANE_BYTES;
    // per-warp staging of the softmax weights of one 32-token tile
    //   VM: fp16 [HPAD][4 k-slot pairs][8 tokens]        otherwise: fp32 pairs [32 tokens][HPAD][2]
    static constexpr int P_WARP_BYTES = VM ? HPAD * 64 : 32 * HPAD * 8;
    static constexpr int Q_BYTES = HPAD * D * 4;              // q' staging during the table build
    static constexpr int P_BYTES = NCW * P_WARP_BYTES > Q_BYTES ? NCW * P_WARP_BYTES : Q_BYTES;
    // Ring stages (each = one page of K and of V).  A consumer warp takes every (NCW/2)-th page; the
    // stage count is a multiple of that stride, so that the page a warp waits for reuses the stage of
    // a page the same warp has already consumed: a waiter is then never more than one mbarrier phase
    // ahead, which the parity test of a phase wait requires.
    static constexpr int STRIDE = NCW / 2;
    static constexpr int NST_FIT = (232448 - 256 - LUT_BYTES - VCB_BYTES - P_BYTES) / (2 * CHUNK);
    static constexpr int NST = (NST_FIT / STRIDE >= 2 ? 2 : 1) * STRIDE;
    static_assert(NCW % 2 == 0 && NST <= NST_FIT, "ring does not fit in shared memory");
    static constexpr int RING_BYTES = NST * 2 * CHUNK;
    static constexpr int OFF_LUT = 0;
    static constexpr int OFF_VCB = OFF_LUT + LUT_BYTES;
    static constexpr int OFF_RING = OFF_VCB + VCB_BYTES;
    static constexpr int OFF_P = OFF_RING + RING_BYTES;
    static constexpr int OFF_BAR = OFF_P + P_BYTES;
    static constexpr int SMEM = OFF_BAR + 256;
    // merge buffer (aliases the table once a segment's scan is done)
    static constexpr int MERGE_ACC_BYTES = NCW * HPAD * D * 4;
    static_assert(MERGE_ACC_BYTES + NCW * HPAD * 8 <= LUT_BYTES, "merge buffer must fit in the table");
    static_assert(SMEM <= 232448, "shared memory budget");
};

__device__ __forceinline__ int clamp_len(int len, int max_pages) {
    const int cap = max_pages * NOVAKV_PAGE_TOKENS;
    return len < 0 ? 0 : (len > cap ? cap : len);
}

// ------------------------------------------------------------------------------------------------
// prepare: query transform + page prefix
// ------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(D)
novakv_prepare_kernel(const __nv_bfloat16* __restrict__ q, const float* __restrict__ rk_inv_t,
                      const int32_t* __restrict__ seq_lens, int batch, int n_q_heads, int n_kv_heads,
                      int max_pages_per_seq, float scale_log2, float* __restrict__ qp,
                      int32_t* __restrict__ page_prefix, uint32_t* __restrict__ dev_status) {
    const int blk = blockIdx.x;
    if (blk == batch * n_q_heads) {
        // exclusive prefix over sequences of (pages * Hkv); small, done by one warp
        if (threadIdx.x < 32) {
            int carry = 0;
            for (int b0 = 0; b0 < batch; b0 += 32) {
                const int b = b0 + threadIdx.x;
                int v = 0;
                if (b < batch) {
                    const int raw = seq_lens[b];
                    const int len = clamp_len(raw, max_pages_per_seq);
                    if (raw != len) atomicOr(dev_status, NOVAKV_DEV_BAD_LENGTH);
                    v = ((len + NOVAKV_PAGE_TOKENS - 1) / NOVAKV_PAGE_TOKENS) * n_kv_heads;
                }
                int incl = v;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t = __shfl_up_sync(0xffffffffu, incl, o);
                    if ((int)threadIdx.x >= o) incl += t;
                }
                if (b < batch) page_prefix[b] = carry + incl - v;
                carry += __shfl_sync(0xffffffffu, incl, 31);
            }
            if (threadIdx.x == 0) page_prefix[batch] = carry;
        }
        return;
    }
    __shared__ float q_s[D];
    const int b = blk / n_q_heads, h = blk - b * n_q_heads;
    const int kvh = h / (n_q_heads / n_kv_heads);
    q_s[threadIdx.x] = __bfloat162float(q[((size_t)b * n_q_heads + h) * D + threadIdx.x]);
    __syncthreads();
    const float* R = rk_inv_t + (size_t)kvh * D * D;
    float acc = 0.f;
#pragma unroll 8
    for (int r = 0; r < D; ++r) acc = fmaf(q_s[r], R[(size_t)r * D + threadIdx.x], acc);
    qp[((size_t)b * n_q_heads + h) * D + threadIdx.x] = acc * scale_log2;
}

// ------------------------------------------------------------------------------------------------
// stage 1 helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void lds_2x64(uint32_t addr, uint64_t& a, uint64_t& b) {
    asm volatile("ld.shared.v2.b64 {%0,%1}, [%2];" : "=l"(a), "=l"(b) : "r"(addr));
}
__device__ __forceinline__ void sts_2x64(uint32_t addr, uint64_t a, uint64_t b) {
    asm volatile("st.shared.v2.b64 [%0], {%1,%2};" ::"r"(addr), "l"(a), "l"(b) : "memory");
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr) {
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds_u128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds_u64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
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

struct Segment {
    int b, kvh, pg0, npg, len;
};

// Locate the (sequence, KV head, page) of global page unit u.  page_prefix is exclusive, length batch+1.
__device__ __forceinline__ Segment locate(const int32_t* __restrict__ page_prefix, const int32_t* __restrict__ seq_lens,
                                          int batch, int n_kv_heads, int max_pages, long u, long u_end) {
    int lo = 0, hi = batch;                    // find b: prefix[b] <= u < prefix[b+1]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((long)page_prefix[mid] <= u) lo = mid; else hi = mid;
    }
    Segment s;
    s.b = lo;
    s.len = clamp_len(seq_lens[lo], max_pages);
    const int pages_b = (s.len + NOVAKV_PAGE_TOKENS - 1) / NOVAKV_PAGE_TOKENS;
    const int rel = (int)(u - page_prefix[lo]);
    s.kvh = rel / pages_b;
    s.pg0 = rel - s.kvh * pages_b;
    const long left = u_end - u;
    s.npg = (int)(left < (long)(pages_b - s.pg0) ? left : (long)(pages_b - s.pg0));
    return s;
}

// ------------------------------------------------------------------------------------------------
// stage 1: persistent index scan
// ------------------------------------------------------------------------------------------------
template <int D, int HG, bool VM>
__global__ void __launch_bounds__(S1_THREADS, 1)
novakv_decode_stage1_kernel(const float* __restrict__ qp, const float* __restrict__ cb_k_lut,
                            const __half* __restrict__ cb_v_img, const uint8_t* __restrict__ k_pages,
                            const uint8_t* __restrict__ v_pages, int n_pages,
                            const int32_t* __restrict__ page_table, int max_pages_per_seq,
                            const int32_t* __restrict__ seq_lens, const int32_t* __restrict__ page_prefix,
                            int batch, int n_q_heads, int n_kv_heads, float* __restrict__ part_ml,
                            float* __restrict__ part_acc, uint32_t* __restrict__ dev_status) {
    using C = S1<D, HG, VM>;
    constexpr int L = C::L, GPS = C::GPS, HPAD = C::HPAD, HSETS = C::HSETS, NST = C::NST, CHUNK = C::CHUNK;
    constexpr int NGB = C::NGB;
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t s_base = smem_u32(smem);
    const uint32_t s_lut = s_base + C::OFF_LUT, s_vcb = s_base + C::OFF_VCB, s_ring = s_base + C::OFF_RING;
    const uint32_t s_p = s_base + C::OFF_P, s_bar = s_base + C::OFF_BAR;
    // barriers: full[NST], empty[NST], vcb
    auto bar_full = [&](int st) { return s_bar + 8u * st; };
    auto bar_empty = [&](int st) { return s_bar + 8u * (NST + st); };
    const uint32_t bar_vcb = s_bar + 8u * (2 * NST);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + C::OFF_BAR + 8 * (2 * NST + 1));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long U = page_prefix[batch];
    const long u_begin = ((long)blockIdx.x * U) / gridDim.x, u_end = ((long)(blockIdx.x + 1) * U) / gridDim.x;
    if (u_begin >= u_end) return;

    if (threadIdx.x == 0) {
        for (int st = 0; st < NST; ++st) { mbar_init(bar_full(st), 2); mbar_init(bar_empty(st), 2); }
        mbar_init(bar_vcb, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();

    // per-warp running state (consumer warps)
    float m_run[HPAD], l_run[HPAD];
    uint64_t acc[HPAD][2];                       // !VM: lane <-> group, 4 value coefficients x HPAD heads
    float macc[HSETS][NGB][4];                   //  VM: lane (r, c): head 4*hs + c, group 8*gb + r, 4 coefficients
#pragma unroll
    for (int h = 0; h < HPAD; ++h) { m_run[h] = M_INIT; l_run[h] = 0.f; acc[h][0] = 0ull; acc[h][1] = 0ull; }
#pragma unroll
    for (int hs = 0; hs < HSETS; ++hs)
#pragma unroll
        for (int gb = 0; gb < NGB; ++gb)
#pragma unroll
            for (int i = 0; i < 4; ++i) macc[hs][gb][i] = 0.f;

    // lane roles of the tensor-core value side (MMA fragment coordinates)
    const int fr = lane >> 2, fc = lane & 3;
    // byte selector that moves byte fc of an index word to bits 8..15 over a slot offset in bits 0..7
    const uint32_t sel_c = 0x5504u | ((uint32_t)fc << 4);
    // B fragments carry a weight in the low or high half depending on the column parity (fr & 1)
    const uint32_t sel_b0 = (fr & 1) ? 0x1044u : 0x4410u, sel_b1 = (fr & 1) ? 0x3244u : 0x4432u;

    int vcb_head = -1;       // KV head whose value codebook is resident
    uint32_t vcb_phase = 0;
    long gp_base = 0;        // pages this CTA has pushed through the ring so far
    long u = u_begin;
    while (u < u_end) {
        const Segment sg = locate(page_prefix, seq_lens, batch, n_kv_heads, max_pages_per_seq, u, u_end);
        const int pair = sg.b * n_kv_heads + sg.kvh;

        // ---- segment prologue -----------------------------------------------------------------
        // q' of this segment's heads -> P area (fp32 [HPAD][D]); heads beyond HG are zero
        for (int i = threadIdx.x; i < HPAD * D; i += S1_THREADS) {
            const int h = i / D, c = i - h * D;
            float v = 0.f;
            if (h < HG) v = qp[((size_t)sg.b * n_q_heads + sg.kvh * HG + h) * D + c];
            reinterpret_cast<float*>(smem + C::OFF_P)[i] = v;
        }
        const bool need_vcb = vcb_head != sg.kvh;
        if (warp == NCW && lane == 0) {
            if (need_vcb) {
                fence_proxy_async();
                mbar_arrive_expect_tx(bar_vcb, VCB_BYTES);
                bulk_g2s(s_vcb, cb_v_img + (size_t)sg.kvh * (VCB_BYTES / 2), VCB_BYTES, bar_vcb);
            }
        }
        __syncthreads();

        if (warp == NCW) {
            // ---- producer warp: stream the segment's pages through the ring --------------------
            // Page ids are fetched 32 at a time (one coalesced load per batch, the next batch in flight
            // while the current one is issued), so that no global-memory latency sits between two bulk
            // copies.
            {
                const int32_t* pt = page_table + (size_t)sg.b * max_pages_per_seq + sg.pg0;
                auto load_ids = [&](int i0) {
                    int page = 0;
                    if (i0 + lane < sg.npg) {
                        page = pt[i0 + lane];
                        if (page < 0 || page >= n_pages) { atomicOr(dev_status, NOVAKV_DEV_BAD_PAGE); page = 0; }
                    }
                    return page;
                };
                int ids_next = load_ids(0);
                bool stop = false;
                // One thread can start a bulk copy only every few hundred clocks, while several lanes of
                // a warp issuing in the same instruction cost little more than one: 2*PG lanes each
                // issue one chunk (K or V) of PG consecutive pages.
                constexpr int PG = NOVAKV_PRODUCER_PAGES;
                const int side = lane & 1;
                for (int i0 = 0; i0 < sg.npg && !stop; i0 += 32) {
                    const int ids = ids_next;
                    ids_next = load_ids(i0 + 32);
                    const int nb = min(32, sg.npg - i0);
                    for (int j = 0; j < nb; j += PG) {
                        const int pj = j + (lane >> 1);
                        const int page = __shfl_sync(0xffffffffu, ids, pj & 31);
                        if (NOVAKV_L2_PREFETCH_PAGES > 0) {
                            // line prefetches into L2, NOVAKV_L2_PREFETCH_PAGES pages ahead of the ring:
                            // one instruction of the warp covers the K and V chunk of one page
                            for (int q = 0; q < PG; ++q) {
                                const int jj = j + q + NOVAKV_L2_PREFETCH_PAGES;
                                const int pf_page = __shfl_sync(0xffffffffu, jj < 32 ? ids : ids_next, jj & 31);
                                if (i0 + jj < sg.npg) {
                                    constexpr int LINES = CHUNK / 128;        // 128-byte lines per chunk: 16 or 8
                                    const size_t off = ((size_t)pf_page * n_kv_heads + sg.kvh) * CHUNK;
                                    const uint8_t* src = (lane < LINES ? k_pages : v_pages) + off + (size_t)(lane % LINES) * 128;
                                    if (lane < 2 * LINES) asm volatile("prefetch.global.L2 [%0];" ::"l"(src));
                                }
                            }
                        }
                        int ok = 1;
                        if (lane < 2 * PG && pj < nb) {
                            const long gp = gp_base + i0 + pj;
                            const int st = (int)(gp % NST);
                            const uint32_t par = (uint32_t)((gp / NST) & 1);
                            if (*abort_flag) {
                                ok = 0;
                            } else if (!mbar_wait_bounded(bar_empty(st), par ^ 1u, abort_flag)) {
                                atomicOr(dev_status, NOVAKV_DEV_WAIT_TIMEOUT);
                                *abort_flag = 1;
                                ok = 0;
                            } else {
                                const size_t off = ((size_t)page * n_kv_heads + sg.kvh) * CHUNK;
                                mbar_arrive_expect_tx(bar_full(st), CHUNK);
                                bulk_g2s(s_ring + st * 2 * CHUNK + side * CHUNK, (side ? v_pages : k_pages) + off, CHUNK, bar_full(st));
                            }
                        }
                        if (!__all_sync(0xffffffffu, ok)) { stop = true; break; }
                    }
                }
            }
        } else {
            // ---- score table: LUT[hs][plane][code][e] (4 heads per entry) ----------------------
            {
                constexpr int CPI = NCW * 2;                                   // codes per iteration (16 entries each)
                const int e = threadIdx.x & 15, code0 = threadIdx.x >> 4;
                const int sigma = e & 7, mpar = e >> 3;
                const float4* cbk = reinterpret_cast<const float4*>(cb_k_lut) + (size_t)sg.kvh * C::PLANES * 256 * 16;
                const float* qs = reinterpret_cast<const float*>(smem + C::OFF_P);
#pragma unroll
                for (int pl = 0; pl < C::PLANES; ++pl) {
                    const int l = sigma * GPS + pl * 2 + mpar;
                    float4 qseg[HPAD];
#pragma unroll
                    for (int h = 0; h < HPAD; ++h) qseg[h] = *reinterpret_cast<const float4*>(qs + h * D + l * 4);
#pragma unroll 4
                    for (int it = 0; it < (256 + CPI - 1) / CPI; ++it) {
                        const int code = code0 + it * CPI;
                        if (code >= 256) break;
                        const float4 cw = cbk[((size_t)pl * 256 + code) * 16 + e];
#pragma unroll
                        for (int hs = 0; hs < HSETS; ++hs) {
                            float4 o;
                            o.x = fmaf(qseg[hs * 4 + 0].w, cw.w, fmaf(qseg[hs * 4 + 0].z, cw.z, fmaf(qseg[hs * 4 + 0].y, cw.y, qseg[hs * 4 + 0].x * cw.x)));
                            o.y = fmaf(qseg[hs * 4 + 1].w, cw.w, fmaf(qseg[hs * 4 + 1].z, cw.z, fmaf(qseg[hs * 4 + 1].y, cw.y, qseg[hs * 4 + 1].x * cw.x)));
                            o.z = fmaf(qseg[hs * 4 + 2].w, cw.w, fmaf(qseg[hs * 4 + 2].z, cw.z, fmaf(qseg[hs * 4 + 2].y, cw.y, qseg[hs * 4 + 2].x * cw.x)));
                            o.w = fmaf(qseg[hs * 4 + 3].w, cw.w, fmaf(qseg[hs * 4 + 3].z, cw.z, fmaf(qseg[hs * 4 + 3].y, cw.y, qseg[hs * 4 + 3].x * cw.x)));
                            *reinterpret_cast<float4*>(smem + C::OFF_LUT + (hs * C::PLANES + pl) * LUT_PLANE_BYTES + code * 256 + e * 16) = o;
                        }
                    }
                }
            }
            // consumer-only barrier: table complete, q' staging no longer needed
            asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory");
            if (need_vcb) {
                if (!mbar_wait_bounded(bar_vcb, vcb_phase, abort_flag)) {
                    atomicOr(dev_status, NOVAKV_DEV_WAIT_TIMEOUT);
                    *abort_flag = 1;
                }
            }

            // ---- consumers: 32-token half pages -----------------------------------------------
            const uint32_t s_pw = s_p + warp * C::P_WARP_BYTES;
            const int q4 = lane >> 3, i8 = lane & 7;
            for (int hp = warp; hp < 2 * sg.npg; hp += NCW) {
                if (*abort_flag) break;
                const int pgi = hp >> 1, half = hp & 1;
                const long gp = gp_base + pgi;
                const int st = (int)(gp % NST);
                const uint32_t par = (uint32_t)((gp / NST) & 1);
                if (!mbar_wait_bounded(bar_full(st), par, abort_flag)) {
                    atomicOr(dev_status, NOVAKV_DEV_WAIT_TIMEOUT);
                    *abort_flag = 1;
                    break;
                }
                const int tok0 = (sg.pg0 + pgi) * NOVAKV_PAGE_TOKENS + half * 32;
                int nvalid = min(32, sg.len - tok0);
#ifdef NOVAKV_EXPERIMENT_SKIP_COMPUTE
                nvalid = 0;     // measurement only: stream the ring without consuming it
#endif
                if (nvalid > 0) {
                    const uint32_t s_k = s_ring + st * 2 * CHUNK + half * 32 * L;
                    const uint32_t s_v = s_ring + st * 2 * CHUNK + CHUNK + half * 2 * (L * NOVAKV_VBLOCK);

                    // ---- key side: lane <-> token, rotate through the 8 slots ----------------
                    uint64_t z[HPAD / 2];
#pragma unroll
                    for (int h = 0; h < HPAD / 2; ++h) z[h] = 0ull;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int sigma = (i8 + q4 + k) & 7;
                        const uint32_t w = GPS == 4 ? lds_u32(s_k + lane * L + sigma * 4) : lds_u16(s_k + lane * L + sigma * 2);
                        const uint32_t sg16 = sigma * 16;
#pragma unroll
                        for (int mm = 0; mm < GPS; ++mm) {
                            // byte mm of w -> bits 8..15, slot offset -> bits 0..7
                            const uint32_t a = __byte_perm(w, sg16, 0x5504 | (mm << 4)) + s_lut + (mm >> 1) * LUT_PLANE_BYTES + (mm & 1) * 128;
#pragma unroll
                            for (int hs = 0; hs < HSETS; ++hs) {
                                uint64_t e01, e23;
                                lds_2x64(a + hs * C::PLANES * LUT_PLANE_BYTES, e01, e23);
                                fadd2(z[hs * 2 + 0], e01);
                                fadd2(z[hs * 2 + 1], e23);
                            }
                        }
                    }
                    // ---- online softmax over the tile (base-2 domain) -------------------------
                    float zf[HPAD];
#pragma unroll
                    for (int h = 0; h < HPAD / 2; ++h) unpack2(z[h], zf[2 * h], zf[2 * h + 1]);
                    bool rescale = false;
                    float alpha[HPAD];
                    __half ph[HPAD];
#pragma unroll
                    for (int h = 0; h < HPAD; ++h) {
                        if (lane >= nvalid) zf[h] = -CUDART_INF_F;
                        const float mx = warp_max(zf[h]);
                        const float m_new = fmaxf(m_run[h], mx);
                        alpha[h] = ex2(m_run[h] - m_new);
                        rescale |= (m_new != m_run[h]);
                        m_run[h] = m_new;
                        zf[h] = ex2(zf[h] - m_new);                 // p
                        if (VM) {
                            // the weight that multiplies the value and the one summed into the normaliser are
                            // the same fp16-rounded number, so the result is an exact softmax of perturbed logits
                            ph[h] = __float2half_rn(zf[h]);
                            zf[h] = __half2float(ph[h]);
                        }
                        l_run[h] = fmaf(l_run[h], alpha[h], zf[h]);
                    }

                    if (!VM) {
                        if (rescale) {
#pragma unroll
                            for (int h = 0; h < HPAD; ++h) {
                                const uint64_t a2 = pack2(alpha[h], alpha[h]);
                                fmul2(acc[h][0], a2);
                                fmul2(acc[h][1], a2);
                            }
                        }
                        __syncwarp();      // previous tile's readers of the P area are done
#pragma unroll
                        for (int h = 0; h < HPAD; h += 2)
                            sts_2x64(s_pw + lane * (HPAD * 8) + h * 8, pack2(zf[h], zf[h]), pack2(zf[h + 1], zf[h + 1]));
                        __syncwarp();

                        // ---- value side on CUDA cores: lane <-> index row (group 8 (row % NGB) + row / NGB) ----
                        constexpr int TPB = D == 128 ? 16 : 8;         // tokens of a 16-token block one lane handles
                        const int hf = D == 128 ? 0 : (lane >> 4), lg = D == 128 ? lane : (lane & 15);
                        const uint32_t l8 = lg * 8;
#pragma unroll
                        for (int blk = 0; blk < 2; ++blk) {
                            const uint4 vb = lds_u128(s_v + blk * (L * NOVAKV_VBLOCK) + lg * 16);
                            uint32_t vw[4] = {vb.x, vb.y, vb.z, vb.w};
                            if (D == 64) { vw[0] = hf ? vb.z : vb.x; vw[1] = hf ? vb.w : vb.y; }
#pragma unroll
                            for (int t = 0; t < TPB; ++t) {
                                const uint32_t a = __byte_perm(vw[t >> 2], l8, 0x5504 | ((t & 3) << 4)) + s_vcb;
                                const uint2 cw = lds_u64(a);
                                const float2 f01 = __half22float2(*reinterpret_cast<const __half2*>(&cw.x));
                                const float2 f23 = __half22float2(*reinterpret_cast<const __half2*>(&cw.y));
                                const uint64_t v01 = pack2(f01.x, f01.y), v23 = pack2(f23.x, f23.y);
                                const uint32_t pa = s_pw + (blk * 16 + hf * 8 + t) * (HPAD * 8);
#pragma unroll
                                for (int h = 0; h < HPAD; h += 2) {
                                    uint64_t p0, p1;
                                    lds_2x64(pa + h * 8, p0, p1);
                                    ffma2(acc[h][0], v01, p0);
                                    ffma2(acc[h][1], v23, p0);
                                    ffma2(acc[h + 1][0], v01, p1);
                                    ffma2(acc[h + 1][1], v23, p1);
                                }
                            }
                        }
                    } else {
                        // ---- value side on tensor cores ---------------------------------------------
                        // D[m][n] += sum_k A[m][k] B[k][n], m16 n8 k16, per 8-token sub-tile and group block gb:
                        //   k = (token j of the sub-tile, sub-coefficient i in {0,1}),
                        //   A[m][(j,i)] = codeword(token j, group 8gb + (m & 7))[2 (m >> 3) + i]      fp16
                        //   B[(j,i)][(h,i')] = p_h(token j) * [i == i']                                fp16
                        //   D[m][(h,i')] = partial of head h, group 8gb + (m & 7), coefficient 2 (m >> 3) + i'
                        if (rescale) {
#pragma unroll
                            for (int hs = 0; hs < HSETS; ++hs) {
                                const float a01 = fc & 1 ? alpha[hs * 4 + 1] : alpha[hs * 4 + 0];
                                const float a23 = fc & 1 ? alpha[hs * 4 + 3] : alpha[hs * 4 + 2];
                                const float al = fc & 2 ? a23 : a01;
#pragma unroll
                                for (int gb = 0; gb < NGB; ++gb)
#pragma unroll
                                    for (int i = 0; i < 4; ++i) macc[hs][gb][i] *= al;
                            }
                        }
                        // weights -> shared memory as fp16, [head][k-slot pair = token & 3][token >> 3, (token >> 2) & 1]
                        __syncwarp();      // previous tile's readers of the P area are done
                        {
                            const uint32_t wa = s_pw + (lane & 3) * 16 + ((lane >> 3) * 2 + ((lane >> 2) & 1)) * 2;
#pragma unroll
                            for (int h = 0; h < HPAD; ++h)
                                asm volatile("st.shared.u16 [%0], %1;" ::"r"(wa + h * 64), "h"(__half_as_ushort(ph[h])) : "memory");
                        }
                        __syncwarp();
                        // B-fragment sources: 8 weights of head (4 hs + fr/2) for the tokens with (token & 3) == fc
                        uint4 pw[HSETS];
#pragma unroll
                        for (int hs = 0; hs < HSETS; ++hs) pw[hs] = lds_u128(s_pw + (hs * 4 + (fr >> 1)) * 64 + fc * 16);

                        // slot of this lane's codeword in the value-codebook row for load x (see the image layout)
                        constexpr int NX = NGB;                      // loads per (sub-tile, token slot): one per group block
#pragma unroll
                        for (int blk = 0; blk < 2; ++blk) {
                            // index rows of this lane's groups for the 16 tokens of the block
                            uint32_t vw[NX][4];
                            uint32_t pos8[NX];
#pragma unroll
                            for (int x = 0; x < NX; ++x) {
                                const int xb4 = (x + fc) & 3;                       // rotated so that a quad hits 4 different slots
                                const int row = fr * NGB + (xb4 % NGB);               // row of group 8 (xb4 % NGB) + fr
                                const uint4 vb = lds_u128(s_v + blk * (L * NOVAKV_VBLOCK) + row * 16);
                                vw[x][0] = vb.x; vw[x][1] = vb.y; vw[x][2] = vb.z; vw[x][3] = vb.w;
                                pos8[x] = (16 * (fr >> 2) + 4 * xb4 + (fr & 3)) * 8;
                            }
#pragma unroll
                            for (int ts = 0; ts < 2; ++ts) {                       // 8-token sub-tiles of the block
                                // gather: X[x][u] = codeword (token 8ts + 4u + fc, group of load x), 2 registers each
                                uint32_t X[NX][2][2];
#pragma unroll
                                for (int x = 0; x < NX; ++x)
#pragma unroll
                                    for (int uu = 0; uu < 2; ++uu) {
                                        const uint32_t a = __byte_perm(vw[x][2 * ts + uu], pos8[x], sel_c) + s_vcb;
                                        const uint2 cw = lds_u64(a);
                                        X[x][uu][0] = cw.x; X[x][uu][1] = cw.y;
                                    }
                                // un-rotate: Y[gb] = X[(gb - fc) mod NX]
                                uint32_t Y[NX][2][2];
                                if (NX == 4) {
                                    uint32_t T[4][2][2];
#pragma unroll
                                    for (int gb = 0; gb < 4; ++gb)
#pragma unroll
                                        for (int uu = 0; uu < 2; ++uu)
#pragma unroll
                                            for (int i = 0; i < 2; ++i) T[gb][uu][i] = (fc & 1) ? X[(gb + 3) & 3][uu][i] : X[gb][uu][i];
#pragma unroll
                                    for (int gb = 0; gb < 4; ++gb)
#pragma unroll
                                        for (int uu = 0; uu < 2; ++uu)
#pragma unroll
                                            for (int i = 0; i < 2; ++i) Y[gb][uu][i] = (fc & 2) ? T[(gb + 2) & 3][uu][i] : T[gb][uu][i];
                                } else {
#pragma unroll
                                    for (int gb = 0; gb < NX; ++gb)
#pragma unroll
                                        for (int uu = 0; uu < 2; ++uu)
#pragma unroll
                                            for (int i = 0; i < 2; ++i) Y[gb][uu][i] = (fc & 1) ? X[(gb + 1) & 1][uu][i] : X[gb][uu][i];
                                }
                                const int t = blk * 2 + ts;                         // sub-tile index within the 32-token tile
#pragma unroll
                                for (int hs = 0; hs < HSETS; ++hs) {
                                    const uint32_t w = t == 0 ? pw[hs].x : (t == 1 ? pw[hs].y : (t == 2 ? pw[hs].z : pw[hs].w));
                                    const uint32_t b0 = __byte_perm(w, 0u, sel_b0), b1 = __byte_perm(w, 0u, sel_b1);
#pragma unroll
                                    for (int gb = 0; gb < NGB; ++gb) {
                                        asm volatile(
                                            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                            : "+f"(macc[hs][gb][0]), "+f"(macc[hs][gb][1]), "+f"(macc[hs][gb][2]), "+f"(macc[hs][gb][3])
                                            : "r"(Y[gb][0][0]), "r"(Y[gb][0][1]), "r"(Y[gb][1][0]), "r"(Y[gb][1][1]), "r"(b0), "r"(b1));
                                    }
                                }
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_empty(st));
            }
        }
        if (need_vcb) { vcb_head = sg.kvh; vcb_phase ^= 1u; }

        // ---- segment epilogue: merge the warps' partials, write one partial ---------------------
        __syncthreads();                                   // scan done everywhere: the table is dead
        float* m_acc = reinterpret_cast<float*>(smem + C::OFF_LUT);                    // [NCW][HPAD][D]
        float* m_ml = reinterpret_cast<float*>(smem + C::OFF_LUT + C::MERGE_ACC_BYTES);  // [NCW][HPAD][2]
        if (warp < NCW) {
#pragma unroll
            for (int h = 0; h < HPAD; ++h) {
                const float lsum = warp_sum(l_run[h]);
                if (lane == 0) { m_ml[(warp * HPAD + h) * 2] = m_run[h]; m_ml[(warp * HPAD + h) * 2 + 1] = lsum; }
                if (!VM) {
                    float a0, a1, a2, a3;
                    unpack2(acc[h][0], a0, a1);
                    unpack2(acc[h][1], a2, a3);
                    if (D == 64) {
                        a0 += __shfl_xor_sync(0xffffffffu, a0, 16);
                        a1 += __shfl_xor_sync(0xffffffffu, a1, 16);
                        a2 += __shfl_xor_sync(0xffffffffu, a2, 16);
                        a3 += __shfl_xor_sync(0xffffffffu, a3, 16);
                    }
                    if (lane < L) {
                        const int g = 8 * (lane % NGB) + lane / NGB;          // group of index row `lane`
                        *reinterpret_cast<float4*>(m_acc + ((size_t)warp * HPAD + h) * D + g * 4) = make_float4(a0, a1, a2, a3);
                    }
                    acc[h][0] = 0ull; acc[h][1] = 0ull;
                }
                m_run[h] = M_INIT; l_run[h] = 0.f;
            }
            if (VM) {
#pragma unroll
                for (int hs = 0; hs < HSETS; ++hs)
#pragma unroll
                    for (int gb = 0; gb < NGB; ++gb) {
                        *reinterpret_cast<float4*>(m_acc + ((size_t)warp * HPAD + hs * 4 + fc) * D + (8 * gb + fr) * 4) =
                            make_float4(macc[hs][gb][0], macc[hs][gb][1], macc[hs][gb][2], macc[hs][gb][3]);
#pragma unroll
                        for (int i = 0; i < 4; ++i) macc[hs][gb][i] = 0.f;
                    }
            }
        }
        __syncthreads();
        {
            const size_t pidx = (size_t)pair + blockIdx.x;      // unique: pair and CTA index both grow along the walk
            for (int i = threadIdx.x; i < HG * D; i += S1_THREADS) {
                const int h = i / D, c = i - h * D;
                float M = M_INIT;
#pragma unroll
                for (int w = 0; w < NCW; ++w) M = fmaxf(M, m_ml[(w * HPAD + h) * 2]);
                float a = 0.f, lsum = 0.f;
#pragma unroll
                for (int w = 0; w < NCW; ++w) {
                    const float sc = ex2(m_ml[(w * HPAD + h) * 2] - M);
                    a = fmaf(sc, m_acc[((size_t)w * HPAD + h) * D + c], a);
                    lsum = fmaf(sc, m_ml[(w * HPAD + h) * 2 + 1], lsum);
                }
                part_acc[(pidx * HG + h) * D + c] = a;
                if (c == 0) { part_ml[(pidx * HG + h) * 2] = M; part_ml[(pidx * HG + h) * 2 + 1] = lsum; }
            }
        }
        __syncthreads();                                   // merge buffer free before the next table build
        gp_base += sg.npg;
        u += sg.npg;
    }

    // fault path only: let copies that were issued but never consumed land before the CTA retires
    if (*abort_flag && threadIdx.x == NCW * 32) {
        for (int st = 0; st < NST; ++st) {
            mbar_wait_bounded(bar_full(st), 0, nullptr, 1ll << 22);
            mbar_wait_bounded(bar_full(st), 1, nullptr, 1ll << 22);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// merge + inverse value transform
// ------------------------------------------------------------------------------------------------
template <int D, int HG>
__global__ void __launch_bounds__(HG * D > 512 ? 512 : HG * D)
novakv_decode_merge_kernel(const float* __restrict__ part_ml, const float* __restrict__ part_acc,
                           const int32_t* __restrict__ page_prefix, const int32_t* __restrict__ seq_lens,
                           int batch, int n_q_heads, int n_kv_heads, int max_pages_per_seq, int grid_s1,
                           const float* __restrict__ rv_t, const float* __restrict__ v_mean,
                           void* __restrict__ out, int out_is_fp32) {
    __shared__ float o_s[HG * D];
    const int pair = blockIdx.x;
    const int b = pair / n_kv_heads, kvh = pair - b * n_kv_heads;
    const int len = clamp_len(seq_lens[b], max_pages_per_seq);
    const int pages_b = (len + NOVAKV_PAGE_TOKENS - 1) / NOVAKV_PAGE_TOKENS;
    const long U = page_prefix[batch];
    for (int i = threadIdx.x; i < HG * D; i += blockDim.x) {
        const int h = i / D, c = i - h * D;
        float val = 0.f;
        if (pages_b > 0) {
            const long u0 = (long)page_prefix[b] + (long)kvh * pages_b, u1 = u0 + pages_b;
            // CTA of unit u: the largest c with floor(c*U/G) <= u
            const int c_first = (int)(((u0 + 1) * grid_s1 - 1) / U), c_last = (int)((u1 * grid_s1 - 1) / U);
            // CTAs in between whose own range is empty wrote nothing: skip them
            float M = M_INIT;
            for (int cta = c_first; cta <= c_last; ++cta) {
                if (((long)cta * U) / grid_s1 >= ((long)(cta + 1) * U) / grid_s1) continue;
                M = fmaxf(M, part_ml[(((size_t)pair + cta) * HG + h) * 2]);
            }
            float a = 0.f, lsum = 0.f;
            for (int cta = c_first; cta <= c_last; ++cta) {
                if (((long)cta * U) / grid_s1 >= ((long)(cta + 1) * U) / grid_s1) continue;
                const size_t pidx = (size_t)pair + cta;
                const float sc = ex2(part_ml[(pidx * HG + h) * 2] - M);
                a = fmaf(sc, part_acc[(pidx * HG + h) * D + c], a);
                lsum = fmaf(sc, part_ml[(pidx * HG + h) * 2 + 1], lsum);
            }
            val = a / lsum;
        }
        o_s[i] = val;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < HG * D; i += blockDim.x) {
        const int h = i / D, r = i - h * D;
        float o = 0.f;
        if (pages_b > 0) {
            const float* R = rv_t + (size_t)kvh * D * D;     // rv_t[c][r] = R_V[r][c]
            float acc = 0.f;
#pragma unroll 8
            for (int c = 0; c < D; ++c) acc = fmaf(o_s[h * D + c], R[(size_t)c * D + r], acc);
            o = acc + v_mean[(size_t)kvh * D + r];
        }
        const size_t oi = ((size_t)b * n_q_heads + kvh * HG + h) * D + r;
        if (out_is_fp32) reinterpret_cast<float*>(out)[oi] = o;
        else reinterpret_cast<__nv_bfloat16*>(out)[oi] = __float2bfloat16_rn(o);
    }
}

// workspace layout
struct WsLayout {
    size_t qp, prefix, ml, acc, total;
};
WsLayout ws_layout(const novakv_ctx* ctx, int batch) {
    auto al = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t d = ctx->cfg.head_dim, hq = ctx->cfg.n_q_heads;
    const size_t n_part = (size_t)batch * ctx->cfg.n_kv_heads + ctx->n_sm;
    WsLayout w;
    w.qp = 0;
    w.prefix = al(w.qp + (size_t)batch * hq * d * 4);
    w.ml = al(w.prefix + ((size_t)batch + 1) * 4);
    w.acc = al(w.ml + n_part * ctx->hg * 2 * 4);
    w.total = al(w.acc + n_part * ctx->hg * d * 4);
    return w;
}

template <int D, int HG, bool VM>
novakv_status launch_decode_t(novakv_ctx* ctx, const novakv_layer& ly, const __nv_bfloat16* q,
                              const uint8_t* k_pages, const uint8_t* v_pages, int n_pages,
                              const int32_t* page_table, int max_pages_per_seq, const int32_t* seq_lens,
                              int batch, float sm_scale, void* out, int out_is_fp32, void* workspace,
                              cudaStream_t stream) {
    using C = S1<D, HG, VM>;
    const WsLayout w = ws_layout(ctx, batch);
    char* ws = (char*)workspace;
    float* qp = (float*)(ws + w.qp);
    int32_t* prefix = (int32_t*)(ws + w.prefix);
    float* part_ml = (float*)(ws + w.ml);
    float* part_acc = (float*)(ws + w.acc);
    const int hq = ctx->cfg.n_q_heads, hkv = ctx->cfg.n_kv_heads;

    novakv_prepare_kernel<D><<<batch * hq + 1, D, 0, stream>>>(q, ly.rk_inv_t, seq_lens, batch, hq, hkv,
        max_pages_per_seq, sm_scale * 1.4426950408889634f, qp, prefix, ctx->dev_status);
    ctx->launches++;

    auto kern = novakv_decode_stage1_kernel<D, HG, VM>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM) != cudaSuccess) return NOVAKV_ECUDA;
    const int grid = ctx->scan_ctas > 0 ? (ctx->scan_ctas < ctx->n_sm ? ctx->scan_ctas : ctx->n_sm) : ctx->n_sm;
    {
        novakv_prof_scope ps(ctx, 0, stream);
        kern<<<grid, S1_THREADS, C::SMEM, stream>>>(qp, ly.cb_k_lut, VM ? ly.cb_v_mma : ly.cb_v_half, k_pages, v_pages, n_pages,
            page_table, max_pages_per_seq, seq_lens, prefix, batch, hq, hkv, part_ml, part_acc, ctx->dev_status);
        ps.end();
        ctx->launches++;
    }
    novakv_decode_merge_kernel<D, HG><<<batch * hkv, (HG * D > 512 ? 512 : HG * D), 0, stream>>>(part_ml, part_acc,
        prefix, seq_lens, batch, hq, hkv, max_pages_per_seq, grid, ly.rv_t, ly.v_mean, out, out_is_fp32);
    ctx->launches++;
    return cudaGetLastError() == cudaSuccess ? NOVAKV_OK : NOVAKV_ECUDA;
}

}  // namespace

size_t novakv_decode_ws_bytes(const novakv_ctx* ctx, int batch) { return ws_layout(ctx, batch).total; }

novakv_status novakv_launch_decode(novakv_ctx* ctx, const novakv_layer& ly, const __nv_bfloat16* q,
    const uint8_t* k_pages, const uint8_t* v_pages, int n_pages, const int32_t* page_table,
    int max_pages_per_seq, const int32_t* seq_lens, int batch, float sm_scale, void* out,
    int out_is_fp32, void* workspace, size_t workspace_bytes, cudaStream_t stream) {
    (void)workspace_bytes;
    const int d = ctx->cfg.head_dim, hg = ctx->hg;
#define NOVAKV_DISPATCH(DD, HH)                                                                             \
    if (d == DD && hg == HH) {                                                                                   \
        if (ctx->value_path == 0)                                                                                \
            return launch_decode_t<DD, HH, false>(ctx, ly, q, k_pages, v_pages, n_pages, page_table,             \
                                                  max_pages_per_seq, seq_lens, batch, sm_scale, out, out_is_fp32, \
                                                  workspace, stream);                                            \
        return launch_decode_t<DD, HH, true>(ctx, ly, q, k_pages, v_pages, n_pages, page_table,                  \
                                             max_pages_per_seq, seq_lens, batch, sm_scale, out, out_is_fp32,     \
                                             workspace, stream);                                                 \
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
