/*
 * CPU oracle for the COD-TDQ hot path: token-group dual-constraint activation
 * quantizer (DSTG + DCRP), static per-output-channel weight quantizer, and the
 * W4A4 linear layer written as an integer contraction plus scaling.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a slow, plain restatement of the
 * paper's definitions, one token-group at a time, in scalar loops.  It shares
 * no code, header, table or constant with the CUDA library, and the CUDA
 * library never calls it.  Only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may load it.
 *
 * What each function follows:
 *   tdq_oracle_quantize_act     Algorithm S1 steps 1-9; Eq. 5, 6, 8-12; the
 *                               numerical conventions of Supp. S4.8 (1e-8 step
 *                               floor, 1e-8 clip floor, population std + 1e-12,
 *                               round-half-to-even) and the rank rule of
 *                               Supp. S2.2 (k = ceil(p*g), 1-indexed).
 *   tdq_oracle_quantize_act_fixed  the same steps 5-9 with a radius fixed beforehand
 *                               (the fixed offline-calibrated control of Supp. S1.2).
 *   tdq_oracle_quantize_weight  Eq. 4 with absmax per-output-channel scales.
 *   tdq_oracle_w4a4_linear      Algorithm S1 step 10 with x_hat = Delta_k * q
 *                               (Eq. 9) and W_hat = s_o * Q_w (Eq. 4) substituted,
 *                               so y[m,o] = s_o * sum_k Delta[m,k] * acc[m,o,k]
 *                               with acc the exact integer dot product of one
 *                               token-group.
 *
 * Precision: every elementwise step of the quantizer is IEEE binary32, in the
 * order the paper writes it (c first, then Delta = c / q_max, then x / Delta).
 * The group mean and standard deviation are accumulated in binary64 and then
 * rounded to binary32.  The linear layer's integer sums are exact; its scaling
 * is done in binary64 and rounded once to binary32.
 *
 * Parity pins (tests marked "not gpu"): Lemma 1 bounds on every group, the
 * rounding-error bound of Proposition 1, zero code <=> |x| <= Delta/2, the
 * worked rank example of Supp. S2.2, brute-force projection on tiny groups,
 * single group == per-tensor absmax quantizer, and the linear layer against a
 * float64 matrix product of the dequantized operands.  The numeric values of
 * codes and scales on the synthetic workloads have no printed counterpart in
 * the paper: for those, "parity unpinned" beyond the properties above.
 *
 * Build:  gcc -O2 -std=c99 -fPIC -shared -fopenmp -ffp-contract=off \
 *             -o libtdq_oracle.so tdq_oracle.c -lm
 * -ffp-contract=off matters: no multiply-add may be fused, or the binary32
 * sequence would no longer be the one written here.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_F32 0
#define ORACLE_BF16 1
#define ORACLE_ENABLE_C1 1u
#define ORACLE_ENABLE_C2 2u
#define ORACLE_POW2_STEP 4u   /* variant: step rounded down to a power of two after the projection */

#define Q_MAX 7
#define Q_MIN (-8)

static float bf16_to_f32(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

static float load_elem(const void* base, int dtype, int64_t idx) {
    if (dtype == ORACLE_BF16) return bf16_to_f32(((const uint16_t*)base)[idx]);
    return ((const float*)base)[idx];
}

static int cmp_float(const void* a, const void* b) {
    float fa = *(const float*)a, fb = *(const float*)b;
    return (fa > fb) - (fa < fb);
}

/* Supp. S2.2: rank k = ceil(frac * g), 1-indexed, kept inside [1, g].  frac is a
 * binary32 number (0.2f is slightly above 0.2), so a product that lands within
 * 1e-6 of an integer is taken to be that integer before the ceiling. */
int32_t tdq_oracle_rank(float frac, int32_t g) {
    double kd = (double)frac * (double)g;
    double kr = floor(kd + 0.5);
    int64_t k = (fabs(kd - kr) < 1e-6) ? (int64_t)kr : (int64_t)ceil(kd);
    if (k < 1) k = 1;
    if (k > g) k = g;
    return (int32_t)k;
}

static uint8_t nibble(int q) { return (uint8_t)(q & 0xF); }

/*
 * Activation quantizer.  x is [M, C] with row stride row_stride (elements).
 * Outputs (each may be NULL):
 *   q      [M, C_pad]      int8 codes, padded channels included
 *   codes  [M, C_pad / 2]  two codes per byte, even channel in the low nibble
 *   scale  [M, K]          Delta_k
 *   clip   [M, K]          c_k after projection and the 1e-8 floor
 *   active [M, K]          0 base radius kept, 1 C1 is the minimum, 2 C2 is the
 *                          minimum (ties resolved base < C1 < C2)
 * Returns 0, or -1 on a bad argument.
 */
int tdq_oracle_quantize_act(const void* x, int x_dtype, int64_t M, int64_t C,
                            int64_t row_stride, int32_t g, float tau, float zr,
                            float p, uint32_t flags, int8_t* q, uint8_t* codes,
                            float* scale, float* clip, uint8_t* active) {
    if (!x || M < 0 || C <= 0 || g <= 0 || (g & 1) || row_stride < C) return -1;
    if (!(zr > 0.0f && zr <= 1.0f) || !(p > 0.0f && p <= 1.0f) || !(tau > 0.0f)) return -1;
    const int64_t K = (C + g - 1) / g;      /* Eq. 5: K = C_pad / g */
    const int64_t C_pad = K * g;
    const int32_t k_base = tdq_oracle_rank(p, g);
    const int32_t k_zr = tdq_oracle_rank(zr, g);
    const float seven_tau = 7.0f * tau;     /* q_max * tau, binary32 */
    int status = 0;

#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        float* xg = (float*)malloc(sizeof(float) * (size_t)g);
        float* ag = (float*)malloc(sizeof(float) * (size_t)g);
        int* qg = (int*)malloc(sizeof(int) * (size_t)g);
        if (!xg || !ag || !qg) {
            status = -1;
            free(xg); free(ag); free(qg);
            continue;
        }
        for (int64_t k = 0; k < K; ++k) {
            /* Alg. S1 steps 1-2: zero-pad to C_pad, take group k. */
            for (int32_t i = 0; i < g; ++i) {
                int64_t ch = k * g + i;
                xg[i] = (ch < C) ? load_elem(x, x_dtype, m * row_stride + ch) : 0.0f;
                ag[i] = fabsf(xg[i]);
            }
            /* mean and population standard deviation in binary64 (step 4(i)). */
            double s = 0.0;
            for (int32_t i = 0; i < g; ++i) s += (double)xg[i];
            double mu = s / (double)g;
            double ss = 0.0;
            for (int32_t i = 0; i < g; ++i) {
                double d = (double)xg[i] - mu;
                ss += d * d;
            }
            float sigma = (float)sqrt(ss / (double)g) + 1e-12f;

            /* order statistics of |x| (steps 3 and 4(ii)). */
            qsort(ag, (size_t)g, sizeof(float), cmp_float);
            float c_base = ag[k_base - 1];   /* k_base == g: the max-abs norm */
            float thr = ag[k_zr - 1];

            /* Eq. 10-12. */
            float c_tau = seven_tau * sigma;
            float c_zr = 14.0f * thr;        /* 2 * q_max * thr */
            float c = c_base;
            uint8_t act = 0;
            if ((flags & ORACLE_ENABLE_C1) && c_tau < c) { c = c_tau; act = 1; }
            if ((flags & ORACLE_ENABLE_C2) && c_zr < c) { c = c_zr; act = 2; }
            if (c < 1e-8f) c = 1e-8f;

            /* Eq. 8 / Alg. S1 step 6. */
            float delta = c / 7.0f;
            if (delta < 1e-8f) delta = 1e-8f;
            if (flags & ORACLE_POW2_STEP) {
                /* not in the paper: Delta' = 2^floor(log2 Delta), c' = 7 Delta' <= c */
                int e;
                (void)frexpf(delta, &e);          /* delta = m * 2^e, m in [0.5, 1) */
                delta = ldexpf(0.5f, e);
                c = 7.0f * delta;
            }

            /* steps 5 and 7. */
            for (int32_t i = 0; i < g; ++i) {
                float xt = xg[i];
                if (xt > c) xt = c;
                if (xt < -c) xt = -c;
                float r = xt / delta;
                float rr = rintf(r);         /* ties to even in the default mode */
                int qi = (int)rr;
                if (qi > Q_MAX) qi = Q_MAX;
                if (qi < Q_MIN) qi = Q_MIN;
                qg[i] = qi;
            }

            if (scale) scale[m * K + k] = delta;
            if (clip) clip[m * K + k] = c;
            if (active) active[m * K + k] = act;
            if (q)
                for (int32_t i = 0; i < g; ++i) q[m * C_pad + k * g + i] = (int8_t)qg[i];
            if (codes)
                for (int32_t i = 0; i < g; i += 2)
                    codes[(m * C_pad + k * g + i) / 2] =
                        (uint8_t)(nibble(qg[i]) | (nibble(qg[i + 1]) << 4));
        }
        free(xg); free(ag); free(qg);
    }
    return status;
}

/*
 * Fixed-radius control (Supp. S1.2, "fixed controls"; Supp. S4.2's fixed offline calibration row):
 * the clip radius is a number fixed beforehand for the whole layer instead of being computed from
 * the activations.  Steps 5-9 of Algorithm S1 with c = max(radius, 1e-8) in every group:
 *   Delta = max(c / 7, 1e-8);  q = clip(rint(clip(x, -c, c) / Delta), -8, 7).
 * Outputs as for tdq_oracle_quantize_act (scale holds the same Delta in every entry).
 */
int tdq_oracle_quantize_act_fixed(const void* x, int x_dtype, int64_t M, int64_t C,
                                  int64_t row_stride, int32_t g, float radius, int8_t* q,
                                  uint8_t* codes, float* scale) {
    if (!x || M < 0 || C <= 0 || g <= 0 || (g & 1) || row_stride < C || !(radius > 0.0f)) return -1;
    const int64_t K = (C + g - 1) / g;
    const int64_t C_pad = K * g;
    float c = radius;
    if (c < 1e-8f) c = 1e-8f;
    float delta = c / 7.0f;
    if (delta < 1e-8f) delta = 1e-8f;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t ch = 0; ch < C_pad; ch += 2) {
            int qi[2];
            for (int j = 0; j < 2; ++j) {
                float xt = (ch + j < C) ? load_elem(x, x_dtype, m * row_stride + ch + j) : 0.0f;
                if (xt > c) xt = c;
                if (xt < -c) xt = -c;
                float rr = rintf(xt / delta);
                int v = (int)rr;
                if (v > Q_MAX) v = Q_MAX;
                if (v < Q_MIN) v = Q_MIN;
                qi[j] = v;
                if (q) q[m * C_pad + ch + j] = (int8_t)v;
            }
            if (codes) codes[(m * C_pad + ch) / 2] = (uint8_t)(nibble(qi[0]) | (nibble(qi[1]) << 4));
        }
        if (scale)
            for (int64_t k = 0; k < K; ++k) scale[m * K + k] = delta;
    }
    return 0;
}

/*
 * Weight quantizer, Eq. 4.  w is [O, I] row-major.  s_o = max(absmax_o / 7, 1e-8).
 * The input dimension is zero-padded to a multiple of pad_to (codes 0).
 *   q      [O, I_pad]      int8, may be NULL
 *   wcodes [O, I_pad / 2]  packed, may be NULL
 *   wscale [O]
 */
int tdq_oracle_quantize_weight(const void* w, int w_dtype, int64_t O, int64_t I,
                               int32_t pad_to, int8_t* q, uint8_t* wcodes,
                               float* wscale) {
    if (!w || O < 0 || I <= 0 || pad_to <= 0 || (pad_to & 1)) return -1;
    const int64_t I_pad = (I + pad_to - 1) / pad_to * pad_to;
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < O; ++o) {
        float amax = 0.0f;
        for (int64_t i = 0; i < I; ++i) {
            float a = fabsf(load_elem(w, w_dtype, o * I + i));
            if (a > amax) amax = a;
        }
        float s = amax / 7.0f;
        if (s < 1e-8f) s = 1e-8f;
        if (wscale) wscale[o] = s;
        for (int64_t i = 0; i < I_pad; i += 2) {
            int qq[2];
            for (int j = 0; j < 2; ++j) {
                float v = (i + j < I) ? load_elem(w, w_dtype, o * I + i + j) : 0.0f;
                int qi = (int)rintf(v / s);
                if (qi > Q_MAX) qi = Q_MAX;
                if (qi < Q_MIN) qi = Q_MIN;
                qq[j] = qi;
                if (q) q[o * I_pad + i + j] = (int8_t)qi;
            }
            if (wcodes) wcodes[(o * I_pad + i) / 2] = (uint8_t)(nibble(qq[0]) | (nibble(qq[1]) << 4));
        }
    }
    return 0;
}

static int unpack_code(const uint8_t* codes, int64_t idx) {
    uint8_t b = codes[idx >> 1];
    int v = (idx & 1) ? (b >> 4) : (b & 0xF);
    return (v >= 8) ? v - 16 : v;           /* two's complement nibble */
}

/*
 * W4A4 linear.  xcodes [M, I_pad/2], xscale [M, K], wcodes [O, I_pad/2],
 * wscale [O], bias [O] or NULL; I_pad = K * g.
 *   acc [M, O, K] int32 (may be NULL): integer dot product of group k
 *   y_d [M, O] double (may be NULL):   s_o * sum_k Delta[m,k] * acc[m,o,k] (+ bias)
 *   y   [M, O] float  (may be NULL):   y_d rounded to binary32
 *   t_abs [M, O] double (may be NULL): s_o * sum_k Delta[m,k] * |acc[m,o,k]|, the size of
 *                the terms that are summed (a diagnostic for tolerances under cancellation;
 *                not part of the method)
 */
int tdq_oracle_w4a4_linear(const uint8_t* xcodes, const float* xscale,
                           const uint8_t* wcodes, const float* wscale,
                           const float* bias, int64_t M, int64_t I_pad, int64_t O,
                           int32_t g, float* y, double* y_d, int32_t* acc, double* t_abs) {
    if (!xcodes || !xscale || !wcodes || !wscale || g <= 0 || I_pad % g) return -1;
    const int64_t K = I_pad / g;
    /* unpack every weight code once; each token row is unpacked once below. */
    int8_t* wq = (int8_t*)malloc((size_t)(O * I_pad) + 1);
    if (!wq) return -1;
    for (int64_t j = 0; j < O * I_pad; ++j) wq[j] = (int8_t)unpack_code(wcodes, j);
    int status = 0;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        int8_t* xq = (int8_t*)malloc((size_t)I_pad + 1);
        if (!xq) { status = -1; continue; }
        for (int64_t j = 0; j < I_pad; ++j) xq[j] = (int8_t)unpack_code(xcodes, m * I_pad + j);
        for (int64_t o = 0; o < O; ++o) {
            double sum = 0.0, sum_abs = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                int32_t a = 0;
                for (int32_t i = 0; i < g; ++i)
                    a += (int32_t)xq[k * g + i] * (int32_t)wq[o * I_pad + k * g + i];
                if (acc) acc[(m * O + o) * K + k] = a;
                sum += (double)xscale[m * K + k] * (double)a;
                sum_abs += (double)xscale[m * K + k] * (double)abs(a);
            }
            if (t_abs) t_abs[m * O + o] = (double)wscale[o] * sum_abs;
            double v = (double)wscale[o] * sum;
            if (bias) v += (double)bias[o];
            if (y_d) y_d[m * O + o] = v;
            if (y) y[m * O + o] = (float)v;
        }
        free(xq);
    }
    free(wq);
    return status;
}

int tdq_oracle_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}
