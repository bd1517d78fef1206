/*
 * CPU oracle for the routed, weight-only-quantized linear layer of MoQE
 * (Mixture of Quantization Experts).
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, obviously-correct C.  Nothing in the
 * CUDA library links, includes or calls this file, and this file includes
 * nothing of the CUDA library.  Only tests, the smoke check and the bench's
 * CPU-baseline leg may load it.
 *
 * What the paper fixes (Section 3.1, "Mixture of Quantization Experts"):
 *   - the experts are several quantized variants of ONE full-precision model,
 *     frozen after construction;
 *   - a router emits one score per expert and each sample (a sequence or an
 *     image) is run by exactly one expert (Section 3.2; Appendix "Convergence
 *     Observations", definition of r(x) in [M]).
 * What it leaves open, and the reading taken here:
 *   - the quantizer: affine round-to-nearest (RTN) per group of g consecutive
 *     input features of one output channel, with the stored fp16 scale used for
 *     the rounding, round-half-to-even, IEEE division;
 *   - asymmetric grids always contain 0 (lo <= 0 <= hi); symmetric grids are
 *     the restricted range [-qmax, qmax] around a fixed zero-point 2^(b-1);
 *   - degenerate groups (scale 0 / non-finite after fp16 rounding) use scale 1;
 *   - routing is a hard arg-max, smallest index wins ties, NaN never wins;
 *   - mixed-expert batches are sorted by expert id with a stable counting sort;
 *   - Y[m][n] = sum_k X[m][k] * dequant(W_e(m))[n][k], accumulated in fp32 in
 *     increasing k, rounded once to bf16.
 *
 * Pins (see tests/test_oracle_*.py): RTN round-trip bound |w - deq| <= s/2,
 * code ranges, closed-form grids that must be recovered exactly, brute-force
 * nearest-code search on small tiles, std::max_element / numpy.argsort(stable)
 * equivalences, exact-integer GEMM cases, single-expert equivalence, batch
 * shuffle invariance, X = I; for the router front end and the load report:
 * brute force in Python, hand-worked examples, sum P = sum F = 1, L_bal = 1 at
 * perfect balance and E at collapse; for the gated pair and the residual add:
 * X = I closed forms, silu(0) = 0, silu(a) - silu(-a) = a, R = 0 and X = 0
 * reductions to the plain product.  The end-to-end numbers of the routed layer have
 * no value printed in the paper: "parity unpinned by the paper" for those;
 * they are pinned by the mathematical properties above instead.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC moqe_oracle.c -lm
 * (-ffp-contract=off: every fp32 operation rounds once, no fused multiply-add.)
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ */
/* storage formats: IEEE binary16 and bfloat16, both round-half-even   */
/* ------------------------------------------------------------------ */
static uint32_t f32_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float bits_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

uint16_t oracle_f32_to_f16(float f)
{
    uint32_t u = f32_bits(f);
    uint32_t sign = (u >> 16) & 0x8000u;
    uint32_t absu = u & 0x7FFFFFFFu;
    if (absu >= 0x7F800000u) {                      /* inf or nan */
        return (uint16_t)(sign | 0x7C00u | ((absu > 0x7F800000u) ? 0x0200u : 0u));
    }
    int32_t exp = (int32_t)(absu >> 23) - 127;      /* unbiased */
    uint32_t man = absu & 0x007FFFFFu;
    if (exp > 15) return (uint16_t)(sign | 0x7C00u); /* certainly overflows */
    if (exp >= -14) {                               /* normal half (before rounding) */
        uint32_t h = ((uint32_t)(exp + 15) << 10) | (man >> 13);
        uint32_t rem = man & 0x1FFFu;
        if (rem > 0x1000u || (rem == 0x1000u && (h & 1u))) h++;   /* may carry into inf: correct */
        return (uint16_t)(sign | h);
    }
    if (exp < -25) return (uint16_t)sign;           /* below half of the smallest subnormal */
    /* subnormal half: value = m * 2^-24, m in [0, 1024) */
    man |= 0x00800000u;
    int shift = -exp - 1;                           /* 14..24: man >> shift has the unit 2^-24 */
    uint32_t h = man >> shift;
    uint32_t rem = man & ((1u << shift) - 1u);
    uint32_t half = 1u << (shift - 1);
    if (rem > half || (rem == half && (h & 1u))) h++;
    return (uint16_t)(sign | h);
}

float oracle_f16_to_f32(uint16_t h)
{
    uint32_t sign = ((uint32_t)h & 0x8000u) << 16;
    uint32_t exp = (h >> 10) & 0x1Fu;
    uint32_t man = h & 0x3FFu;
    if (exp == 0x1Fu) return bits_f32(sign | 0x7F800000u | (man << 13));
    if (exp == 0) {
        float v = (float)man * 5.9604644775390625e-08f;     /* man * 2^-24, exact */
        return sign ? -v : v;
    }
    return bits_f32(sign | ((exp + 112u) << 23) | (man << 13));
}

uint16_t oracle_f32_to_bf16(float f)
{
    uint32_t u = f32_bits(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

float oracle_bf16_to_f32(uint16_t b) { return bits_f32((uint32_t)b << 16); }

/* ------------------------------------------------------------------ */
/* Expert construction: RTN quantizer (reading of Section 3.1)          */
/* ------------------------------------------------------------------ */
/*
 * W [N][K] fp32 -> codes [N][K] (one code per byte), scales/zeros [N][K/g]
 * as fp16 bit patterns.  group == 0 means g = K (one group per output channel).
 * Returns 0, or -1 on a bad argument.
 */
int oracle_quantize_rtn(const float *W, int N, int K, int bits, int group, int sym,
                        uint8_t *codes, uint16_t *scales_f16, uint16_t *zeros_f16)
{
    if (!W || !codes || !scales_f16 || !zeros_f16) return -1;
    if (N <= 0 || K <= 0 || bits < 2 || bits > 8) return -1;
    int g = (group == 0) ? K : group;
    if (g <= 0 || K % g != 0) return -1;
    int G = K / g;
    const int32_t L = (1 << bits) - 1;              /* largest code */
    const int32_t half = 1 << (bits - 1);           /* symmetric zero-point */
    const int32_t qmax = half - 1;

    for (int n = 0; n < N; ++n) {
        for (int gi = 0; gi < G; ++gi) {
            const float *w = W + (size_t)n * K + (size_t)gi * g;
            uint8_t *c = codes + (size_t)n * K + (size_t)gi * g;
            float s32;
            int32_t z;
            if (sym) {
                float a = 0.0f;
                for (int k = 0; k < g; ++k) { float v = fabsf(w[k]); if (v > a) a = v; }
                s32 = a / (float)qmax;
            } else {
                float lo = 0.0f, hi = 0.0f;
                for (int k = 0; k < g; ++k) { if (w[k] < lo) lo = w[k]; if (w[k] > hi) hi = w[k]; }
                s32 = (hi - lo) / (float)L;
            }
            uint16_t sh = oracle_f32_to_f16(s32);
            float s = oracle_f16_to_f32(sh);
            if (!(s > 0.0f) || isinf(s)) { sh = 0x3C00u; s = 1.0f; }   /* degenerate group */
            if (sym) {
                z = half;
                for (int k = 0; k < g; ++k) {
                    int32_t q = (int32_t)rintf(w[k] / s);
                    if (q < -qmax) q = -qmax;
                    if (q > qmax) q = qmax;
                    c[k] = (uint8_t)(q + half);
                }
            } else {
                float lo = 0.0f;
                for (int k = 0; k < g; ++k) if (w[k] < lo) lo = w[k];
                z = (int32_t)rintf(-lo / s);
                if (z < 0) z = 0;
                if (z > L) z = L;
                for (int k = 0; k < g; ++k) {
                    int32_t q = (int32_t)rintf(w[k] / s) + z;
                    if (q < 0) q = 0;
                    if (q > L) q = L;
                    c[k] = (uint8_t)q;
                }
            }
            scales_f16[(size_t)n * G + gi] = sh;
            zeros_f16[(size_t)n * G + gi] = oracle_f32_to_f16((float)z);   /* exact: z <= 255 */
        }
    }
    return 0;
}

/* Explicit dequantization to fp32: w^ = float(s) * float(int(c) - int(z)).
 * The product of an 11-bit and a <=9-bit significand is exact in fp32. */
int oracle_dequantize(const uint8_t *codes, const uint16_t *scales_f16, const uint16_t *zeros_f16,
                      int N, int K, int group, float *What)
{
    if (!codes || !scales_f16 || !zeros_f16 || !What || N <= 0 || K <= 0) return -1;
    int g = (group == 0) ? K : group;
    if (g <= 0 || K % g != 0) return -1;
    int G = K / g;
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            size_t gi = (size_t)n * G + k / g;
            float s = oracle_f16_to_f32(scales_f16[gi]);
            int32_t z = (int32_t)oracle_f16_to_f32(zeros_f16[gi]);
            int32_t c = (int32_t)codes[(size_t)n * K + k];
            What[(size_t)n * K + k] = s * (float)(c - z);
        }
    return 0;
}

/* ------------------------------------------------------------------ */
/* Hard routing: one expert per sample (Section 3.2; r(x) in [M])       */
/* ------------------------------------------------------------------ */
int oracle_route(const float *logits, int S, int E, int32_t *ids)
{
    if (!logits || !ids || S < 0 || E <= 0) return -1;
    for (int s = 0; s < S; ++s) {
        const float *l = logits + (size_t)s * E;
        int best = -1;
        float bv = 0.0f;
        for (int e = 0; e < E; ++e) {
            float v = l[e];
            if (isnan(v)) continue;                 /* NaN never wins */
            if (best < 0 || v > bv) { best = e; bv = v; }
        }
        ids[s] = (best < 0) ? 0 : best;             /* all-NaN row -> expert 0 */
    }
    return 0;
}

/* Per-sample ids -> per-row ids: rows [off[s], off[s+1]) belong to sample s. */
int oracle_expand_ids(const int32_t *ids, const int32_t *row_offsets, int S, int32_t *row_ids)
{
    if (!ids || !row_offsets || !row_ids || S < 0) return -1;
    for (int s = 0; s < S; ++s)
        for (int32_t r = row_offsets[s]; r < row_offsets[s + 1]; ++r) row_ids[r] = ids[s];
    return 0;
}

/* ------------------------------------------------------------------ */
/* Stable counting sort of rows by expert id                            */
/* ------------------------------------------------------------------ */
/* counts[E], offsets[E+1] (exclusive scan), perm[M] = source row of sorted slot
 * j, inv[M] with inv[perm[j]] = j.  n_i = counts[i] is the per-expert sample
 * count of the paper's load statistic F_i = n_i / B (Section 3.3).
 * Returns -2 if an id lies outside [0, E). */
int oracle_permutation(const int32_t *row_ids, int M, int E,
                       int32_t *counts, int32_t *offsets, int32_t *perm, int32_t *inv)
{
    if (!row_ids || !counts || !offsets || !perm || M < 0 || E <= 0) return -1;
    for (int e = 0; e < E; ++e) counts[e] = 0;
    for (int m = 0; m < M; ++m) {
        if (row_ids[m] < 0 || row_ids[m] >= E) return -2;
        counts[row_ids[m]]++;
    }
    offsets[0] = 0;
    for (int e = 0; e < E; ++e) offsets[e + 1] = offsets[e] + counts[e];
    int32_t *cursor = (int32_t *)malloc(sizeof(int32_t) * (size_t)E);
    if (!cursor) return -1;
    for (int e = 0; e < E; ++e) cursor[e] = offsets[e];
    for (int m = 0; m < M; ++m) {
        int32_t j = cursor[row_ids[m]]++;
        perm[j] = m;
        if (inv) inv[m] = j;
    }
    free(cursor);
    return 0;
}

/* Xp[j][:] = X[perm[j]][:]  (rows of C 16-bit elements) */
int oracle_permute_rows(const uint16_t *X, const int32_t *perm, int M, int C, uint16_t *Xp)
{
    if (!X || !perm || !Xp || M < 0 || C <= 0) return -1;
    for (int j = 0; j < M; ++j)
        memcpy(Xp + (size_t)j * C, X + (size_t)perm[j] * C, sizeof(uint16_t) * (size_t)C);
    return 0;
}

/* Y[perm[j]][:] = Yp[j][:] */
int oracle_unpermute_rows(const uint16_t *Yp, const int32_t *perm, int M, int C, uint16_t *Y)
{
    if (!Yp || !perm || !Y || M < 0 || C <= 0) return -1;
    for (int j = 0; j < M; ++j)
        memcpy(Y + (size_t)perm[j] * C, Yp + (size_t)j * C, sizeof(uint16_t) * (size_t)C);
    return 0;
}

/* ------------------------------------------------------------------ */
/* Routed GEMM: each row is multiplied by ITS expert's dequantized W    */
/* ------------------------------------------------------------------ */
/*
 * X bf16 [M][K]; row_ids[M]; What[e] = fp32 [N][K] dequantized weight of expert e.
 * rows == NULL: all M rows, Y is [M][N].  Otherwise rows[R] lists the rows to
 * compute and Y is [R][N] (sampling for the large workloads).
 * Y_bf16 and/or Y_f32 (the unrounded fp32 accumulator) may be NULL.
 * Accumulation: fp32, k increasing, product rounded then added (no FMA).
 */
int oracle_routed_gemm(const uint16_t *X, const int32_t *row_ids, int M, int K, int N, int E,
                       const float *const *What, const int32_t *rows, int R,
                       uint16_t *Y_bf16, float *Y_f32)
{
    if (!X || !row_ids || !What || M < 0 || K <= 0 || N <= 0 || E <= 0) return -1;
    int nrows = rows ? R : M;
    for (int i = 0; i < nrows; ++i) {
        int m = rows ? rows[i] : i;
        if (m < 0 || m >= M) return -1;
        if (row_ids[m] < 0 || row_ids[m] >= E) return -2;
    }
    long total = (long)nrows * N;
#pragma omp parallel
    {
        float *xf = (float *)malloc(sizeof(float) * (size_t)K);
        int cached = -1;
#pragma omp for schedule(static)
        for (long t = 0; t < total; ++t) {
            int i = (int)(t / N), n = (int)(t % N);
            int m = rows ? rows[i] : i;
            if (cached != i) {
                for (int k = 0; k < K; ++k) xf[k] = oracle_bf16_to_f32(X[(size_t)m * K + k]);
                cached = i;
            }
            const float *w = What[row_ids[m]] + (size_t)n * K;
            float acc = 0.0f;
            for (int k = 0; k < K; ++k) acc += xf[k] * w[k];
            if (Y_f32) Y_f32[(size_t)i * N + n] = acc;
            if (Y_bf16) Y_bf16[(size_t)i * N + n] = oracle_f32_to_bf16(acc);
        }
        free(xf);
    }
    return 0;
}

/* Same product accumulated in fp64 (every fp32*fp32 product is exact in fp64):
 * used only to show how far the fp32 accumulation above is from the exact sum. */
int oracle_routed_gemm_f64(const uint16_t *X, const int32_t *row_ids, int M, int K, int N, int E,
                           const float *const *What, const int32_t *rows, int R, double *Y_f64)
{
    if (!X || !row_ids || !What || !Y_f64 || M < 0 || K <= 0 || N <= 0 || E <= 0) return -1;
    int nrows = rows ? R : M;
    for (int i = 0; i < nrows; ++i) {
        int m = rows ? rows[i] : i;
        if (m < 0 || m >= M) return -1;
        if (row_ids[m] < 0 || row_ids[m] >= E) return -2;
    }
    long total = (long)nrows * N;
#pragma omp parallel for schedule(static)
    for (long t = 0; t < total; ++t) {
        int i = (int)(t / N), n = (int)(t % N);
        int m = rows ? rows[i] : i;
        const float *w = What[row_ids[m]] + (size_t)n * K;
        const uint16_t *x = X + (size_t)m * K;
        double acc = 0.0;
        for (int k = 0; k < K; ++k) acc += (double)oracle_bf16_to_f32(x[k]) * (double)w[k];
        Y_f64[t] = acc;
    }
    return 0;
}

/* ---------------------------------------------------------------------------
 * Router front end.  Section 3.2 ("Router Model"): the router ends in an MLP that maps
 * the sample's feature vector to one score per expert, and one expert index leaves it.
 * The stand-in here (the paper's trained routers are not available): the feature
 * vector of a sample is the mean of its rows; the MLP is two layers with a ReLU
 * between them and no biases.  Everything in fp64:
 *   pooled[s][h] = (1 / n_s) * sum_{rows r of sample s} X[r][h]
 *   hidden[s][d] = max(0, sum_h pooled[s][h] * W1[d][h])
 *   logits[s][e] = sum_d hidden[s][d] * W2[e][d]
 * A sample without rows has pooled = 0.
 * ------------------------------------------------------------------------- */
int oracle_router_mlp(const uint16_t *X, const int32_t *row_offsets, int S, int H, const float *W1, int D,
                      const float *W2, int E, double *pooled, double *logits)
{
    if (!X || !row_offsets || !W1 || !W2 || !logits || S < 0 || H <= 0 || D <= 0 || E <= 0) return -1;
    double *pool = (double *)malloc(sizeof(double) * (size_t)H);
    double *hid = (double *)malloc(sizeof(double) * (size_t)D);
    if (!pool || !hid) { free(pool); free(hid); return -1; }
    for (int s = 0; s < S; ++s) {
        int r0 = row_offsets[s], r1 = row_offsets[s + 1];
        if (r1 < r0) { free(pool); free(hid); return -1; }
        for (int h = 0; h < H; ++h) {
            double acc = 0.0;
            for (int r = r0; r < r1; ++r) acc += (double)oracle_bf16_to_f32(X[(size_t)r * H + h]);
            pool[h] = r1 > r0 ? acc / (double)(r1 - r0) : 0.0;
            if (pooled) pooled[(size_t)s * H + h] = pool[h];
        }
        for (int d = 0; d < D; ++d) {
            double acc = 0.0;
            for (int h = 0; h < H; ++h) acc += pool[h] * (double)W1[(size_t)d * H + h];
            hid[d] = acc > 0.0 ? acc : 0.0;
        }
        for (int e = 0; e < E; ++e) {
            double acc = 0.0;
            for (int d = 0; d < D; ++d) acc += hid[d] * (double)W2[(size_t)e * D + d];
            logits[(size_t)s * E + e] = acc;
        }
    }
    free(pool);
    free(hid);
    return 0;
}

/* Load report of a routed batch.  Section 3.3 ("Router Fine-Tuning"), the balance term of the
 * objective, evaluated at inference time on the batch's S samples (the paper's B) and E experts (its N):
 *   p_i(x) = softmax(logits(x))_i,  P_i = (1/S) sum_x p_i(x),  F_i = n_i / S,  L_bal = E * sum_i P_i * F_i
 * with n_i the number of samples dispatched to expert i (ids).  fp64. */
int oracle_load_report(const double *logits, const int32_t *ids, int S, int E, double *P, double *F, double *Lbal)
{
    if (!logits || !ids || !P || !F || !Lbal || S <= 0 || E <= 0) return -1;
    for (int e = 0; e < E; ++e) { P[e] = 0.0; F[e] = 0.0; }
    for (int s = 0; s < S; ++s) {
        if (ids[s] < 0 || ids[s] >= E) return -2;
        const double *l = logits + (size_t)s * E;
        double mx = l[0];
        for (int e = 1; e < E; ++e) if (l[e] > mx) mx = l[e];
        double den = 0.0;
        for (int e = 0; e < E; ++e) den += exp(l[e] - mx);
        for (int e = 0; e < E; ++e) P[e] += exp(l[e] - mx) / den;
        F[ids[s]] += 1.0;
    }
    double lb = 0.0;
    for (int e = 0; e < E; ++e) { P[e] /= (double)S; F[e] /= (double)S; lb += P[e] * F[e]; }
    *Lbal = (double)E * lb;
    return 0;
}

/* ---------------------------------------------------------------------------
 * Steps either side of the routed product inside an expert's forward pass (Section 4.4 times whole expert
 * forwards, so what sits between two linear layers counts).  Both use the routed product above -- fp32,
 * k increasing, product rounded then added -- and round to bf16 ONCE at the end:
 *   gated pair   : Y[m][n] = bf16( silu(a) * b ),  a = (X . Wgate_e^T)[m][n],  b = (X . Wup_e^T)[m][n],
 *                  silu(a) = a / (1 + exp(-a)) in fp32
 *   residual add : Y[m][n] = bf16( a + float(R[m][n]) ),  R bf16
 * ------------------------------------------------------------------------- */
int oracle_routed_gated_pair(const uint16_t *X, const int32_t *row_ids, int M, int K, int N, int E,
                             const float *const *Wgate, const float *const *Wup, uint16_t *Y_bf16)
{
    if (!X || !row_ids || !Wgate || !Wup || !Y_bf16 || M < 0 || K <= 0 || N <= 0 || E <= 0) return -1;
    for (int m = 0; m < M; ++m)
        if (row_ids[m] < 0 || row_ids[m] >= E) return -2;
    long total = (long)M * N;
#pragma omp parallel for schedule(static)
    for (long t = 0; t < total; ++t) {
        int m = (int)(t / N), n = (int)(t % N);
        const float *wg = Wgate[row_ids[m]] + (size_t)n * K;
        const float *wu = Wup[row_ids[m]] + (size_t)n * K;
        const uint16_t *x = X + (size_t)m * K;
        float a = 0.0f, b = 0.0f;
        for (int k = 0; k < K; ++k) {
            float xf = oracle_bf16_to_f32(x[k]);
            a += xf * wg[k];
            b += xf * wu[k];
        }
        float silu = a / (1.0f + expf(-a));
        Y_bf16[t] = oracle_f32_to_bf16(silu * b);
    }
    return 0;
}

int oracle_routed_gemm_residual(const uint16_t *X, const int32_t *row_ids, int M, int K, int N, int E,
                                const float *const *What, const uint16_t *R, uint16_t *Y_bf16)
{
    if (!X || !row_ids || !What || !R || !Y_bf16 || M < 0 || K <= 0 || N <= 0 || E <= 0) return -1;
    for (int m = 0; m < M; ++m)
        if (row_ids[m] < 0 || row_ids[m] >= E) return -2;
    long total = (long)M * N;
#pragma omp parallel for schedule(static)
    for (long t = 0; t < total; ++t) {
        int m = (int)(t / N), n = (int)(t % N);
        const float *w = What[row_ids[m]] + (size_t)n * K;
        const uint16_t *x = X + (size_t)m * K;
        float acc = 0.0f;
        for (int k = 0; k < K; ++k) acc += oracle_bf16_to_f32(x[k]) * w[k];
        Y_bf16[t] = oracle_f32_to_bf16(acc + oracle_bf16_to_f32(R[t]));
    }
    return 0;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
