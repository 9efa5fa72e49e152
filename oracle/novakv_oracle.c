/*
 * NOVA-KV CPU oracle (TEST INFRASTRUCTURE ONLY).
 *
 * A plain, slow, float64 restatement of what the decode and append paths compute, written
 * from the paper.  It is used by the tests, by the smoke check and by the benchmark's CPU
 * baseline; the product path never calls it.  It shares no code with the CUDA library.
 *
 *   encode  : Algorithm 1 line 7 and Sec. 2.2 ("Quantization"): coefficients
 *             r = (k - kbar) R_K, s = (v - vbar) R_V, then per group of g coefficients the
 *             index of the nearest codeword (exact Euclidean search, App. B "Calibration").
 *   decode  : Sec. 2.2 reconstruction k^ = Q(r) R_K^{-1} + kbar (Theorem 1 text), v^ = Q(s) R_V^T
 *             + vbar (Corollary 1), followed by textbook attention, Eq. "scores":
 *             softmax(q k^T / sqrt(d)) v.  Keys and values are dequantised EXPLICITLY; the
 *             query fold, the dropped mean (Lemma S1) and the transform-domain value
 *             accumulation used on the GPU are deliberately NOT used here.
 *   R_K^{-1} is taken from the stored synthesis matrix: R_K^{-1} = (R_K^{-T})^T.
 *
 * Precision: everything is float64.  The encoder is the paper's exact Euclidean nearest-neighbour
 * search (Sec. 2.2 "Quantization"; App. B "Calibration"): float64 coefficients, float64 squared
 * distances, codewords visited in ascending index, the first minimum kept (lowest index wins an
 * exact tie).  Beside the index the oracle reports the float64 relative gap (d2 - d1) / d1 between
 * the two smallest distances, which is how near-ties are counted.  Two stored formats define some
 * of their bits through binary32 arithmetic (the per-token key scale and the scalar INT2 value
 * codec, see below); there the binary32 step is part of the format's definition and is stated with
 * the function.
 *
 * Pins (tests/test_oracle_pins.py): exact invariance of the attention products when the
 * quantiser is the identity, generalised Parseval relation (Prop. 1), Lemma S1, one-token
 * and equal-logit caches, brute force against an independently written search, hand-built
 * tie cases, split invariance, planted needle; for the scaled key format: power-of-two
 * equivariance, unit RMS of the normalised coefficients, reduction to the unscaled encoder at
 * rho = 1, linearity of the reconstruction in rho, the paper's bit-rate arithmetic.  No
 * end-to-end numeric value is printed in the paper, so the numeric end-to-end parity is pinned
 * by those identities only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <float.h>

typedef struct {
    int n_kv_heads, head_dim, group_size, codebook_size;
    const double* rk;        /* [Hkv][d][d]  analysis  R_K            */
    const double* rk_inv_t;  /* [Hkv][d][d]  R_K^{-T}                 */
    const double* rv;        /* [Hkv][d][d]  R_V (orthogonal)         */
    const double* k_mean;    /* [Hkv][d]                              */
    const double* v_mean;    /* [Hkv][d]                              */
    const double* cb_k;      /* [Hkv][L][C][g]                        */
    const double* cb_v;      /* [Hkv][L][C][g]                        */
} oracle_tables;

/* row vector times matrix: y[c] = sum_r x[r] M[r][c] */
static void rowvec_mat(const double* x, const double* m, int d, double* y)
{
    for (int c = 0; c < d; ++c) y[c] = 0.0;
    for (int r = 0; r < d; ++r)
        for (int c = 0; c < d; ++c) y[c] += x[r] * m[r * d + c];
}

/* row vector times transposed matrix: y[r] = sum_c x[c] M[r][c] */
static void rowvec_mat_t(const double* x, const double* m, int d, double* y)
{
    for (int r = 0; r < d; ++r) {
        double s = 0.0;
        for (int c = 0; c < d; ++c) s += x[c] * m[r * d + c];
        y[r] = s;
    }
}

/* Transform coefficients of one vector: (x - mean) M. */
void oracle_coefficients(const double* x, const double* mean, const double* m, int d, double* out)
{
    double* xc = (double*)malloc(sizeof(double) * d);
    for (int i = 0; i < d; ++i) xc[i] = x[i] - mean[i];
    rowvec_mat(xc, m, d, out);
    free(xc);
}

/*
 * Nearest-codeword search for one group (Sec. 2.2 "Quantization": the encoder returns the index of
 * the nearest codeword; App. B "Calibration": exact Euclidean search; lowest index wins ties).
 * coef: g float64 coefficients.  cb: [C][g] float64.  Returns the index of the first minimum of the
 * float64 squared distance; *gap gets the relative gap (d2 - d1) / d1 between the two smallest
 * distances (DBL_MAX if d1 == 0 and d2 > 0, 0 if both are 0).
 */
static int search_group(const double* coef, const double* cb, int g, int C, double* gap)
{
    double d1 = DBL_MAX, d2 = DBL_MAX;
    int best = -1;
    for (int c = 0; c < C; ++c) {
        const double* cw = cb + (long)c * g;
        double s = 0.0;
        for (int i = 0; i < g; ++i) {
            double e = coef[i] - cw[i];
            s += e * e;
        }
        if (best < 0 || s < d1) { d2 = d1; d1 = s; best = c; }
        else if (s < d2) { d2 = s; }
    }
    if (gap) *gap = (d1 > 0.0) ? (d2 - d1) / d1 : (d2 > 0.0 ? DBL_MAX : 0.0);
    return best;
}

/*
 * Encode from coefficients that are already given (float64 holding the values to search).
 * coef: [n][d]; cb: [L][C][g]; idx: [n][L].  gap may be NULL.
 */
void oracle_search(const double* coef, long n, int d, int g, int C, const double* cb,
                   uint8_t* idx, double* gap)
{
    int L = d / g;
#pragma omp parallel for schedule(static)
    for (long j = 0; j < n; ++j) {
        for (int l = 0; l < L; ++l) {
            double gp;
            idx[j * L + l] = (uint8_t)search_group(coef + j * d + l * g, cb + (long)l * C * g, g, C, &gp);
            if (gap) gap[j * L + l] = gp;
        }
    }
}

/*
 * Write path for n tokens: k, v [n][Hkv][d] -> kidx, vidx [n][Hkv][L] (+ gap arrays of the same
 * shape, may be NULL).
 */
void oracle_encode(const oracle_tables* t, const double* k, const double* v, long n,
                   uint8_t* kidx, uint8_t* vidx, double* kgap, double* vgap)
{
    const int d = t->head_dim, g = t->group_size, C = t->codebook_size, H = t->n_kv_heads;
    const int L = d / g;
#pragma omp parallel for collapse(2) schedule(static)
    for (long j = 0; j < n; ++j) {
        for (int h = 0; h < H; ++h) {
            double* coef = (double*)malloc(sizeof(double) * d);
            long o = (j * H + h);
            /* keys */
            oracle_coefficients(k + o * d, t->k_mean + (long)h * d, t->rk + (long)h * d * d, d, coef);
            for (int l = 0; l < L; ++l) {
                double gp;
                kidx[o * L + l] = (uint8_t)search_group(coef + l * g, t->cb_k + ((long)h * L + l) * C * g, g, C, &gp);
                if (kgap) kgap[o * L + l] = gp;
            }
            /* values */
            oracle_coefficients(v + o * d, t->v_mean + (long)h * d, t->rv + (long)h * d * d, d, coef);
            for (int l = 0; l < L; ++l) {
                double gp;
                vidx[o * L + l] = (uint8_t)search_group(coef + l * g, t->cb_v + ((long)h * L + l) * C * g, g, C, &gp);
                if (vgap) vgap[o * L + l] = gp;
            }
            free(coef);
        }
    }
}

/* Dequantise one key: r^ = concat_l cb_k[l][idx[l]];  k^ = r^ (R_K^{-T})^T + kbar. */
static void reconstruct_key(const oracle_tables* t, int h, const uint8_t* idx, double* out)
{
    const int d = t->head_dim, g = t->group_size, C = t->codebook_size, L = d / g;
    double* r = (double*)malloc(sizeof(double) * d);
    for (int l = 0; l < L; ++l)
        for (int i = 0; i < g; ++i)
            r[l * g + i] = t->cb_k[(((long)h * L + l) * C + idx[l]) * g + i];
    rowvec_mat_t(r, t->rk_inv_t + (long)h * d * d, d, out);   /* r (R_K^{-T})^T = r R_K^{-1} */
    for (int i = 0; i < d; ++i) out[i] += t->k_mean[(long)h * d + i];
    free(r);
}

/* Dequantise one value: s^ = concat_l cb_v[l][idx[l]];  v^ = s^ R_V^T + vbar. */
static void reconstruct_value(const oracle_tables* t, int h, const uint8_t* idx, double* out)
{
    const int d = t->head_dim, g = t->group_size, C = t->codebook_size, L = d / g;
    double* s = (double*)malloc(sizeof(double) * d);
    for (int l = 0; l < L; ++l)
        for (int i = 0; i < g; ++i)
            s[l * g + i] = t->cb_v[(((long)h * L + l) * C + idx[l]) * g + i];
    rowvec_mat_t(s, t->rv + (long)h * d * d, d, out);         /* s R_V^T */
    for (int i = 0; i < d; ++i) out[i] += t->v_mean[(long)h * d + i];
    free(s);
}

/* kidx, vidx: [S][Hkv][L] -> k_hat, v_hat: [S][Hkv][d] */
void oracle_reconstruct(const oracle_tables* t, const uint8_t* kidx, const uint8_t* vidx, long S,
                        double* k_hat, double* v_hat)
{
    const int d = t->head_dim, H = t->n_kv_heads, L = d / t->group_size;
#pragma omp parallel for collapse(2) schedule(static)
    for (long j = 0; j < S; ++j)
        for (int h = 0; h < H; ++h) {
            long o = j * H + h;
            if (k_hat) reconstruct_key(t, h, kidx + o * L, k_hat + o * d);
            if (v_hat) reconstruct_value(t, h, vidx + o * L, v_hat + o * d);
        }
}

/*
 * Textbook single-query attention over explicit keys and values (Eq. "scores"):
 * q: [Hq][d];  k, v: [S][Hkv][d];  out: [Hq][d].  Query head h reads KV head h / (Hq/Hkv).
 */
void oracle_attention(const double* q, const double* k, const double* v, long S, int Hq, int Hkv,
                      int d, double sm_scale, double* out)
{
    const int hg = Hq / Hkv;
#pragma omp parallel for schedule(static)
    for (int h = 0; h < Hq; ++h) {
        const int kv = h / hg;
        double* z = (double*)malloc(sizeof(double) * (S > 0 ? S : 1));
        double zmax = -DBL_MAX;
        for (long j = 0; j < S; ++j) {
            const double* kj = k + (j * Hkv + kv) * d;
            double s = 0.0;
            for (int i = 0; i < d; ++i) s += q[(long)h * d + i] * kj[i];
            z[j] = s * sm_scale;
            if (z[j] > zmax) zmax = z[j];
        }
        double den = 0.0;
        for (long j = 0; j < S; ++j) { z[j] = exp(z[j] - zmax); den += z[j]; }
        for (int i = 0; i < d; ++i) out[(long)h * d + i] = 0.0;
        for (long j = 0; j < S; ++j) {
            const double p = z[j] / den;
            const double* vj = v + (j * Hkv + kv) * d;
            for (int i = 0; i < d; ++i) out[(long)h * d + i] += p * vj[i];
        }
        free(z);
    }
}

/*
 * Decode step for one sequence: dequantise the whole cache, then textbook attention.
 * q: [Hq][d]; kidx, vidx: [S][Hkv][L]; out: [Hq][d].  S == 0 gives zeros.
 */
void oracle_decode(const oracle_tables* t, const double* q, const uint8_t* kidx,
                   const uint8_t* vidx, long S, int Hq, double sm_scale, double* out)
{
    const int d = t->head_dim, H = t->n_kv_heads;
    if (S <= 0) { memset(out, 0, sizeof(double) * (size_t)Hq * d); return; }
    double* k_hat = (double*)malloc(sizeof(double) * (size_t)S * H * d);
    double* v_hat = (double*)malloc(sizeof(double) * (size_t)S * H * d);
    oracle_reconstruct(t, kidx, vidx, S, k_hat, v_hat);
    oracle_attention(q, k_hat, v_hat, S, Hq, H, d, sm_scale, out);
    free(k_hat);
    free(v_hat);
}

/* ------------------------------------------------------------------------------------------------
 * Key format with a per-token scale (Algorithm "Codebook training", the "Normalize" step; App. B
 * "Decoding kernel and read path": the read side takes rho_j from per-token metadata and applies it
 * with a single multiply; Sec. 5 "Bit rate": a BF16 scale per token, 16/128 = 0.125 bit/elem).
 *
 *   rho_j = ||r_j||_2 / sqrt(d),   r_j <- r_j / rho_j   before the codebook search,
 *   k^_j  = rho_j * Q(r_j / rho_j) R_K^{-1} + kbar       on the read side.
 *
 * Where floating point decides stored bits the arithmetic is the one the library boundary
 * documents: r is the binary32-rounded coefficient vector; the sum of squares is accumulated
 * in binary64; rho = sqrt(sum / d) in binary64, rounded to binary32 and then to bfloat16
 * (round to nearest even both times); a scale that is not a positive finite number is replaced
 * by 1; the normalised coefficient is the binary32 quotient r_i / rho.
 * ---------------------------------------------------------------------------------------------- */
static float bf16_round(float x)
{
    uint32_t u;
    memcpy(&u, &x, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) return x;          /* inf / nan unchanged */
    u += 0x7fffu + ((u >> 16) & 1u);                          /* round to nearest, ties to even */
    u &= 0xffff0000u;
    memcpy(&x, &u, 4);
    return x;
}

/* coef: d float64 coefficients.  Returns rho (a bfloat16 value held in a float) and writes the
 * normalised coefficients (binary32 values held in float64) to out. */
float oracle_key_scale(const double* coef, int d, double* out)
{
    double ss = 0.0;
    for (int i = 0; i < d; ++i) {
        const double r = (double)(float)coef[i];
        ss += r * r;
    }
    float rho = bf16_round((float)sqrt(ss / (double)d));
    if (!(rho > 0.f) || !isfinite(rho)) rho = 1.f;
    for (int i = 0; i < d; ++i) out[i] = (double)((float)coef[i] / rho);
    return rho;
}

/* Write path with the key scale: as oracle_encode, plus kscale [n][Hkv] (bfloat16 values as float). */
void oracle_encode_scaled(const oracle_tables* t, const double* k, const double* v, long n,
                          uint8_t* kidx, uint8_t* vidx, float* kscale, double* kgap, double* vgap)
{
    const int d = t->head_dim, g = t->group_size, C = t->codebook_size, H = t->n_kv_heads;
    const int L = d / g;
#pragma omp parallel for collapse(2) schedule(static)
    for (long j = 0; j < n; ++j) {
        for (int h = 0; h < H; ++h) {
            double* coef = (double*)malloc(sizeof(double) * d);
            double* nrm = (double*)malloc(sizeof(double) * d);
            long o = (j * H + h);
            oracle_coefficients(k + o * d, t->k_mean + (long)h * d, t->rk + (long)h * d * d, d, coef);
            kscale[o] = oracle_key_scale(coef, d, nrm);
            for (int l = 0; l < L; ++l) {
                double gp;
                kidx[o * L + l] = (uint8_t)search_group(nrm + l * g, t->cb_k + ((long)h * L + l) * C * g, g, C, &gp);
                if (kgap) kgap[o * L + l] = gp;
            }
            oracle_coefficients(v + o * d, t->v_mean + (long)h * d, t->rv + (long)h * d * d, d, coef);
            for (int l = 0; l < L; ++l) {
                double gp;
                vidx[o * L + l] = (uint8_t)search_group(coef + l * g, t->cb_v + ((long)h * L + l) * C * g, g, C, &gp);
                if (vgap) vgap[o * L + l] = gp;
            }
            free(coef);
            free(nrm);
        }
    }
}

/* Dequantise one scaled key: r^ = rho * concat_l cb_k[l][idx[l]];  k^ = r^ R_K^{-1} + kbar. */
static void reconstruct_key_scaled(const oracle_tables* t, int h, const uint8_t* idx, double rho, double* out)
{
    const int d = t->head_dim, g = t->group_size, C = t->codebook_size, L = d / g;
    double* r = (double*)malloc(sizeof(double) * d);
    for (int l = 0; l < L; ++l)
        for (int i = 0; i < g; ++i)
            r[l * g + i] = rho * t->cb_k[(((long)h * L + l) * C + idx[l]) * g + i];
    rowvec_mat_t(r, t->rk_inv_t + (long)h * d * d, d, out);
    for (int i = 0; i < d; ++i) out[i] += t->k_mean[(long)h * d + i];
    free(r);
}

/* kidx, vidx: [S][Hkv][L], kscale [S][Hkv] -> k_hat, v_hat: [S][Hkv][d] */
void oracle_reconstruct_scaled(const oracle_tables* t, const uint8_t* kidx, const uint8_t* vidx,
                               const float* kscale, long S, double* k_hat, double* v_hat)
{
    const int d = t->head_dim, H = t->n_kv_heads, L = d / t->group_size;
#pragma omp parallel for collapse(2) schedule(static)
    for (long j = 0; j < S; ++j)
        for (int h = 0; h < H; ++h) {
            long o = j * H + h;
            if (k_hat) reconstruct_key_scaled(t, h, kidx + o * L, (double)kscale[o], k_hat + o * d);
            if (v_hat) reconstruct_value(t, h, vidx + o * L, v_hat + o * d);
        }
}

/* Decode step of one sequence on the scaled-key cache: explicit dequantisation, textbook attention. */
void oracle_decode_scaled(const oracle_tables* t, const double* q, const uint8_t* kidx,
                          const uint8_t* vidx, const float* kscale, long S, int Hq, double sm_scale,
                          double* out)
{
    const int d = t->head_dim, H = t->n_kv_heads;
    if (S <= 0) { memset(out, 0, sizeof(double) * (size_t)Hq * d); return; }
    double* k_hat = (double*)malloc(sizeof(double) * (size_t)S * H * d);
    double* v_hat = (double*)malloc(sizeof(double) * (size_t)S * H * d);
    oracle_reconstruct_scaled(t, kidx, vidx, kscale, S, k_hat, v_hat);
    oracle_attention(q, k_hat, v_hat, S, Hq, H, d, sm_scale, out);
    free(k_hat);
    free(v_hat);
}

/* ------------------------------------------------------------------------------------------------
 * Learned attention sink (App. "Attention sinks in the quantized serving path"): an extra logit
 * s_h per query head that enters the softmax normaliser but has no value vector,
 *     p_j = exp(z_j) / ( sum_i exp(z_i) + exp(s_h) ),   o = sum_j p_j v_j,
 * with z_j the full logits q.k_j * sm_scale (the oracle dequantises keys explicitly, mean included,
 * so the offset correction the GPU applies to the sink logit has no counterpart here).
 * sink: [Hq] natural-log units.  S == 0 gives zeros (all the mass sits on the sink).
 * ---------------------------------------------------------------------------------------------- */
void oracle_attention_sink(const double* q, const double* k, const double* v, long S, int Hq, int Hkv,
                           int d, double sm_scale, const double* sink, double* out)
{
    const int hg = Hq / Hkv;
#pragma omp parallel for schedule(static)
    for (int h = 0; h < Hq; ++h) {
        const int kv = h / hg;
        double* z = (double*)malloc(sizeof(double) * (S > 0 ? S : 1));
        double zmax = sink[h];
        for (long j = 0; j < S; ++j) {
            const double* kj = k + (j * Hkv + kv) * d;
            double s = 0.0;
            for (int i = 0; i < d; ++i) s += q[(long)h * d + i] * kj[i];
            z[j] = s * sm_scale;
            if (z[j] > zmax) zmax = z[j];
        }
        double den = exp(sink[h] - zmax);
        for (long j = 0; j < S; ++j) { z[j] = exp(z[j] - zmax); den += z[j]; }
        for (int i = 0; i < d; ++i) out[(long)h * d + i] = 0.0;
        for (long j = 0; j < S; ++j) {
            const double p = z[j] / den;
            const double* vj = v + (j * Hkv + kv) * d;
            for (int i = 0; i < d; ++i) out[(long)h * d + i] += p * vj[i];
        }
        free(z);
    }
}

/* Decode step with a sink: explicit dequantisation (kscale may be NULL: unscaled key format). */
void oracle_decode_sink(const oracle_tables* t, const double* q, const uint8_t* kidx, const uint8_t* vidx,
                        const float* kscale, long S, int Hq, double sm_scale, const double* sink, double* out)
{
    const int d = t->head_dim, H = t->n_kv_heads;
    if (S <= 0) { memset(out, 0, sizeof(double) * (size_t)Hq * d); return; }
    double* k_hat = (double*)malloc(sizeof(double) * (size_t)S * H * d);
    double* v_hat = (double*)malloc(sizeof(double) * (size_t)S * H * d);
    if (kscale) oracle_reconstruct_scaled(t, kidx, vidx, kscale, S, k_hat, v_hat);
    else oracle_reconstruct(t, kidx, vidx, S, k_hat, v_hat);
    oracle_attention_sink(q, k_hat, v_hat, S, Hq, H, d, sm_scale, sink, out);
    free(k_hat);
    free(v_hat);
}

/* ------------------------------------------------------------------------------------------------
 * Scalar value codec of the deployed format (Sec. 5 "Bit rate": values are 2-bit integers with one BF16
 * scale and one BF16 zero-point per token, 2 + 32/128 = 2.25 bits per element; App. B read path: the
 * codes are dequantised in a rotation basis), in the Corollary 1 basis R_V:
 *     s = (v - vbar) R_V,   code_i = clamp(round((s_i - zero) / scale), 0, 3),
 *     s^_i = zero + scale * code_i,   v^ = s^ R_V^T + vbar,
 * one (scale, zero) pair per token and KV head.  Where floating point decides stored bits the
 * arithmetic is the one the library boundary documents: s is the binary32-rounded coefficient
 * vector; zero = bf16(min_i s_i); scale = bf16((max_i s_i - zero) / 3) evaluated in binary32, replaced
 * by 1 if it is not positive and finite; code_i = clamp(rint((s_i - zero) / scale), 0, 3) with the
 * subtraction and the division in binary32 and ties to even.
 * ---------------------------------------------------------------------------------------------- */
void oracle_int2_quantise(const double* coef, int d, uint8_t* codes, float* scale_out, float* zero_out)
{
    float mn = (float)coef[0], mx = (float)coef[0];
    for (int i = 1; i < d; ++i) {
        const float s = (float)coef[i];
        if (s < mn) mn = s;
        if (s > mx) mx = s;
    }
    const float zero = bf16_round(mn);
    float scale = bf16_round((mx - zero) / 3.0f);
    if (!(scale > 0.f) || !isfinite(scale)) scale = 1.f;
    for (int i = 0; i < d; ++i) {
        const float t = (float)coef[i] - zero;
        float u = rintf(t / scale);
        if (!(u > 0.f)) u = 0.f;
        if (u > 3.f) u = 3.f;
        codes[i] = (uint8_t)u;
    }
    *scale_out = scale;
    *zero_out = zero;
}

/* Values of n tokens -> codes [n][Hkv][d] (one code per byte, 0..3) and meta [n][Hkv][2] = (scale, zero). */
void oracle_encode_values_int2(const oracle_tables* t, const double* v, long n, uint8_t* codes, float* meta)
{
    const int d = t->head_dim, H = t->n_kv_heads;
#pragma omp parallel for collapse(2) schedule(static)
    for (long j = 0; j < n; ++j)
        for (int h = 0; h < H; ++h) {
            double* coef = (double*)malloc(sizeof(double) * d);
            long o = j * H + h;
            oracle_coefficients(v + o * d, t->v_mean + (long)h * d, t->rv + (long)h * d * d, d, coef);
            oracle_int2_quantise(coef, d, codes + o * d, meta + o * 2, meta + o * 2 + 1);
            free(coef);
        }
}

/* codes [S][Hkv][d], meta [S][Hkv][2] -> v_hat [S][Hkv][d] */
void oracle_reconstruct_values_int2(const oracle_tables* t, const uint8_t* codes, const float* meta, long S,
                                    double* v_hat)
{
    const int d = t->head_dim, H = t->n_kv_heads;
#pragma omp parallel for collapse(2) schedule(static)
    for (long j = 0; j < S; ++j)
        for (int h = 0; h < H; ++h) {
            long o = j * H + h;
            double* s = (double*)malloc(sizeof(double) * d);
            for (int i = 0; i < d; ++i) s[i] = (double)meta[o * 2 + 1] + (double)meta[o * 2] * (double)codes[o * d + i];
            rowvec_mat_t(s, t->rv + (long)h * d * d, d, v_hat + o * d);
            for (int i = 0; i < d; ++i) v_hat[o * d + i] += t->v_mean[(long)h * d + i];
            free(s);
        }
}
