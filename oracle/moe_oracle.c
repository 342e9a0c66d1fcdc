/*
 * CPU oracle for one decode step of the routed Mixture-of-Experts operator with
 * block-wise FP8 weights.  TEST INFRASTRUCTURE ONLY: it exists so that the CUDA
 * library can be checked against something written straight from the paper.
 * It is deliberately plain and slow (double accumulators, no blocking, no
 * fusion, no SIMD) and shares no code, header, table or helper with the CUDA
 * path.  Only tests, the smoke check and the benchmark's cpu-baseline leg may
 * call it.
 *
 * The operator (Section 3, "MonoMoE Design": top-k/quantize, up-projection,
 * down-projection, reduce; Section 4.1: E4M3 weights and activations, 128x128
 * weight block scales, 128-element activation groups) is an encoding pipeline,
 * so the oracle takes its steps in the paper's order:
 *
 *   1. router logits  L[t,e] = sum_h X[t,h]*Wr[e,h]                (Section 3.3, router-logit overlap)
 *   2. scores: softmax over all E, or sigmoid (+ selection bias)   (Section 4.1, routing policies)
 *   3. top-k by key, ties to the lowest expert index
 *   4. routing weights, optionally renormalised over the selected, times routed_scale
 *   5. input quantisation per token per `group` columns to E4M3    (Section 4.1)
 *   6. gate/up projection with per-(block,group) scale products    (Eq. 9, weight-major form)
 *   7. SiLU(gate)*up, rounded to fp32                              (Section 3.3, up-projection epilogue)
 *   8. requantisation of the intermediate exactly as step 5        (same passage)
 *   9. down projection                                             (Section 3.2/3.3)
 *  10. out[t] = bf16( sum over slots in slot order of w*y )        (Section 3.2, final weighted reduction)
 *
 * Precision.  Sums are accumulated in double.  Every value the method stores in
 * a narrower type is rounded to exactly that type: activation scales and the
 * scaled values are fp32 (IEEE division), codes are E4M3 by round-to-nearest-
 * even with saturation at +-448, routing weights are fp32, the output is bf16
 * rounded once from the double sum.  The quantisation decisions are taken in
 * fp32 because that is the precision the method itself quantises in.
 *
 * Readings where the paper is silent: gate = rows [0,I) of W13, up = rows
 * [I,2I); amax floor 1e-10; scale = amax/448 by true division; the routing
 * weight multiplies after the down projection; slots are ordered by
 * (key descending, index ascending).
 *
 * Parity status: the codec, the routing, the quantisation and the whole
 * operator are pinned by closed forms, hand-worked cases, a dense float64
 * re-evaluation on tiny shapes and invariants (tests/test_oracle_*.py).
 * Agreement with the authors' own kernel is "parity unpinned": the paper prints
 * no output value of the operator for any input.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_SCORE_SOFTMAX 0
#define ORACLE_SCORE_SIGMOID_BIAS 1

/* ---- scalar codecs -------------------------------------------------------- */

/* bf16 -> double: the 16 bits are the upper half of an IEEE fp32. */
double oracle_bf16_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* double -> bf16, one round-to-nearest-even to an 8-bit significand. */
uint16_t oracle_double_to_bf16(double x) {
    uint16_t sign = (uint16_t)(signbit(x) ? 0x8000u : 0u);
    double a = fabs(x);
    if (isnan(x)) return (uint16_t)(sign | 0x7FC0u);
    if (a == 0.0) return sign;
    if (isinf(a)) return (uint16_t)(sign | 0x7F80u);
    if (a < ldexp(1.0, -126)) {                 /* subnormal range: units of 2^-133 */
        double n = rint(ldexp(a, 133));         /* 0..128; 128 is the smallest normal */
        return (uint16_t)(sign | (uint16_t)n);
    }
    int e;
    double m = frexp(a, &e);                    /* a = m*2^e, m in [0.5,1) */
    m *= 2.0; e -= 1;                           /* m in [1,2) */
    double n = rint(m * 128.0);                 /* 128..256, ties to even */
    if (n == 256.0) { n = 128.0; e += 1; }
    if (e > 127) return (uint16_t)(sign | 0x7F80u);
    return (uint16_t)(sign | ((uint16_t)(e + 127) << 7) | ((uint16_t)n - 128u));
}

/* E4M3 ("e4m3fn": 1-4-3, bias 7, no infinity, NaN = 0x7F/0xFF, max 448) -> double. */
double oracle_e4m3_to_double(uint8_t c) {
    int s = c >> 7, e = (c >> 3) & 0xF, m = c & 7;
    double v;
    if (e == 0xF && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return s ? -v : v;
}

/* fp32 -> E4M3, round-to-nearest-even, finite overflow saturates to +-448. */
uint8_t oracle_e4m3_from_float(float v) {
    uint8_t s = (uint8_t)(signbit(v) ? 0x80u : 0u);
    float a = fabsf(v);
    if (isnan(v)) return (uint8_t)(s | 0x7Fu);
    if (a > 448.0f) return (uint8_t)(s | 0x7Eu);
    if (a < 0.015625f) {                        /* below 2^-6: subnormal step 2^-9 */
        float n = rintf(a * 512.0f);            /* exact scaling, ties to even, 0..8 */
        return (uint8_t)(s | (uint8_t)n);       /* n == 8 is the smallest normal 0x08 */
    }
    int e;
    float m = frexpf(a, &e);
    m *= 2.0f; e -= 1;                          /* a = m*2^e, m in [1,2) */
    float n = rintf(m * 8.0f);                  /* 8..16 */
    if (n == 16.0f) { n = 8.0f; e += 1; }
    return (uint8_t)(s | (uint8_t)((e + 7) << 3) | ((uint8_t)n - 8u));
}

/* ---- step 5 / 8: group quantisation --------------------------------------- */

/* Quantise `n` fp32 values (n a multiple of group) into E4M3 bytes and one fp32 scale per group. */
void oracle_quantize_groups(const float* x, int n, int group, uint8_t* q, float* scale) {
    for (int g = 0; g < n / group; ++g) {
        float amax = 0.0f;
        for (int i = 0; i < group; ++i) {
            float a = fabsf(x[g * group + i]);
            if (a > amax) amax = a;
        }
        if (amax < 1e-10f) amax = 1e-10f;
        volatile float s = amax / 448.0f;       /* fp32 division, kept in fp32 */
        scale[g] = s;
        for (int i = 0; i < group; ++i) {
            volatile float r = x[g * group + i] / s;
            q[g * group + i] = oracle_e4m3_from_float(r);
        }
    }
}

/* ---- steps 1-4: routing ---------------------------------------------------- */

static void route_token(int H, int E, int K, int scoring, int renorm, float routed_scale,
                        const uint16_t* x, const uint16_t* Wr, const float* bias,
                        int32_t* ids, float* w, double* margin, float* logits_out) {
    double* L = (double*)malloc(sizeof(double) * (size_t)E);
    double* key = (double*)malloc(sizeof(double) * (size_t)E);
    double* val = (double*)malloc(sizeof(double) * (size_t)E);
    char* taken = (char*)calloc((size_t)E, 1);
    for (int e = 0; e < E; ++e) {
        double acc = 0.0;
        for (int h = 0; h < H; ++h)
            acc += oracle_bf16_to_double(x[h]) * oracle_bf16_to_double(Wr[(size_t)e * H + h]);
        L[e] = acc;
        if (logits_out) logits_out[e] = (float)acc;
    }
    if (scoring == ORACLE_SCORE_SOFTMAX) {
        double mx = L[0], sum = 0.0;
        for (int e = 1; e < E; ++e) if (L[e] > mx) mx = L[e];
        for (int e = 0; e < E; ++e) { val[e] = exp(L[e] - mx); sum += val[e]; }
        for (int e = 0; e < E; ++e) { val[e] /= sum; key[e] = L[e]; }
    } else {
        for (int e = 0; e < E; ++e) {
            val[e] = 1.0 / (1.0 + exp(-L[e]));
            key[e] = val[e] + (bias ? (double)bias[e] : 0.0);
        }
    }
    double kth = 0.0;
    for (int j = 0; j < K; ++j) {               /* repeated arg-max, strict '>' keeps the lowest index */
        int best = -1;
        for (int e = 0; e < E; ++e)
            if (!taken[e] && (best < 0 || key[e] > key[best])) best = e;
        taken[best] = 1;
        ids[j] = best;
        kth = key[best];
    }
    if (margin) {
        if (K == E) *margin = INFINITY;
        else {
            int best = -1;
            for (int e = 0; e < E; ++e)
                if (!taken[e] && (best < 0 || key[e] > key[best])) best = e;
            *margin = kth - key[best];
        }
    }
    double denom = 1.0;
    if (renorm) {
        denom = 0.0;
        for (int j = 0; j < K; ++j) denom += val[ids[j]];
    }
    for (int j = 0; j < K; ++j) w[j] = (float)(val[ids[j]] / denom * (double)routed_scale);
    free(L); free(key); free(val); free(taken);
}

/* ---- the operator ----------------------------------------------------------- */

/*
 * All arrays are host memory, row-major, caller-owned.  `group` is both the
 * activation group width and the weight block edge (128 in the method; smaller
 * values only make tiny brute-force tests possible).  `expert_map`, if not
 * NULL, maps an expert id to its index in compacted weight arrays (-1: absent;
 * selecting an absent expert returns -2).  If `ids_in`/`w_in` are not NULL the
 * routing steps are skipped and these are used (fixed-routing experiments,
 * Section 4.2).  Optional outputs may be NULL.
 * Returns 0, or a negative value for invalid arguments.
 */
int moe_oracle(int T, int H, int E, int I, int K, int scoring, int renorm, float routed_scale, int group,
               const uint16_t* hidden_bf16, const uint16_t* Wr_bf16, const float* bias,
               const int32_t* expert_map,
               const uint8_t* W13q, const float* W13s, const uint8_t* W2q, const float* W2s,
               const int32_t* ids_in, const float* w_in,
               uint16_t* out_bf16, int32_t* ids, float* w, double* margin, float* logits,
               uint8_t* xq, float* xs, float* act, uint8_t* hq, float* hs,
               double* y_slots, double* out_f64) {
    if (T < 0 || H <= 0 || E <= 0 || I <= 0 || K <= 0 || K > E || group <= 0) return -1;
    if (H % group || I % group) return -1;
    if (!ids || !w || !xq || !xs || !out_bf16) return -1;
    const int HG = H / group, IG = I / group;
    const size_t w13_rows = (size_t)2 * I, w13_sr = (size_t)(2 * I / group);

    /* steps 1-4 */
    for (int t = 0; t < T; ++t) {
        if (ids_in && w_in) {
            for (int j = 0; j < K; ++j) { ids[t * K + j] = ids_in[t * K + j]; w[t * K + j] = w_in[t * K + j]; }
            if (margin) margin[t] = INFINITY;
        } else {
            route_token(H, E, K, scoring, renorm, routed_scale, hidden_bf16 + (size_t)t * H, Wr_bf16, bias,
                        ids + t * K, w + t * K, margin ? margin + t : NULL, logits ? logits + (size_t)t * E : NULL);
        }
    }
    /* step 5 */
    {
        float* xf = (float*)malloc(sizeof(float) * (size_t)H);
        for (int t = 0; t < T; ++t) {
            for (int h = 0; h < H; ++h) xf[h] = (float)oracle_bf16_to_double(hidden_bf16[(size_t)t * H + h]);
            oracle_quantize_groups(xf, H, group, xq + (size_t)t * H, xs + (size_t)t * HG);
        }
        free(xf);
    }
    for (int p = 0; p < T * K; ++p) {
        int e = ids[p];
        if (e < 0 || e >= E) return -1;
        if (expert_map && expert_map[e] < 0) return -2;
    }

    int status = 0;
    double* yall = (double*)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1) * K * H);
    #pragma omp parallel for schedule(dynamic)
    for (int p = 0; p < T * K; ++p) {
        const int t = p / K;
        const int e = ids[p];
        const size_t ew = (size_t)(expert_map ? expert_map[e] : e);
        const uint8_t* A13 = W13q + ew * w13_rows * (size_t)H;
        const float* S13 = W13s + ew * w13_sr * (size_t)HG;
        const uint8_t* A2 = W2q + ew * (size_t)H * I;
        const float* S2 = W2s + ew * (size_t)HG * IG;
        const uint8_t* xqt = xq + (size_t)t * H;
        const float* xst = xs + (size_t)t * HG;

        double* g = (double*)malloc(sizeof(double) * 2 * (size_t)I);
        float* a = (float*)malloc(sizeof(float) * (size_t)I);
        uint8_t* hq_p = (uint8_t*)malloc((size_t)I);
        float* hs_p = (float*)malloc(sizeof(float) * (size_t)IG);
        double* xd = (double*)malloc(sizeof(double) * (size_t)H);
        for (int h = 0; h < H; ++h) xd[h] = oracle_e4m3_to_double(xqt[h]);

        /* step 6: gate/up rows j < 2I */
        for (int j = 0; j < 2 * I; ++j) {
            double acc = 0.0;
            for (int kb = 0; kb < HG; ++kb) {
                double blk = 0.0;
                for (int h = kb * group; h < (kb + 1) * group; ++h)
                    blk += oracle_e4m3_to_double(A13[(size_t)j * H + h]) * xd[h];
                acc += blk * ((double)S13[(size_t)(j / group) * HG + kb] * (double)xst[kb]);
            }
            g[j] = acc;
        }
        /* step 7: SwiGLU, materialised in fp32 */
        for (int i = 0; i < I; ++i) {
            double z = g[i];
            double silu = z / (1.0 + exp(-z));
            a[i] = (float)(silu * g[I + i]);
        }
        /* step 8: requantise */
        oracle_quantize_groups(a, I, group, hq_p, hs_p);
        if (act) memcpy(act + (size_t)p * I, a, sizeof(float) * (size_t)I);
        if (hq) memcpy(hq + (size_t)p * I, hq_p, (size_t)I);
        if (hs) memcpy(hs + (size_t)p * IG, hs_p, sizeof(float) * (size_t)IG);
        /* step 9: down projection rows r < H */
        for (int r = 0; r < H; ++r) {
            double acc = 0.0;
            for (int ib = 0; ib < IG; ++ib) {
                double blk = 0.0;
                for (int i = ib * group; i < (ib + 1) * group; ++i)
                    blk += oracle_e4m3_to_double(A2[(size_t)r * I + i]) * oracle_e4m3_to_double(hq_p[i]);
                acc += blk * ((double)S2[(size_t)(r / group) * IG + ib] * (double)hs_p[ib]);
            }
            yall[(size_t)p * H + r] = acc;
        }
        free(g); free(a); free(hq_p); free(hs_p); free(xd);
    }
    /* step 10: weighted reduction in slot order, one rounding to bf16 */
    for (int t = 0; t < T; ++t)
        for (int r = 0; r < H; ++r) {
            double acc = 0.0;
            for (int j = 0; j < K; ++j) acc += (double)w[t * K + j] * yall[((size_t)t * K + j) * H + r];
            if (out_f64) out_f64[(size_t)t * H + r] = acc;
            out_bf16[(size_t)t * H + r] = oracle_double_to_bf16(acc);
        }
    if (y_slots) memcpy(y_slots, yall, sizeof(double) * (size_t)T * K * H);
    free(yall);
    return status;
}

/* Number of worker threads the expert loop will use (1 when built without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int moe_oracle_threads(void) { return omp_get_max_threads(); }
void moe_oracle_set_threads(int n) { if (n > 0) omp_set_num_threads(n); }
#else
int moe_oracle_threads(void) { return 1; }
void moe_oracle_set_threads(int n) { (void)n; }
#endif
