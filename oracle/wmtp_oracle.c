/*
 * CPU oracle for draft decode attention -- TEST INFRASTRUCTURE, not part of the product.
 *
 * Plain fp64 softmax attention, written as the definition reads (Section 4 "Mechanism":
 * the draft attends over a key set; Appendix D: o = sum_j p_j v_j with p the softmax of
 * the scaled logits).  Two passes per head: logits and their maximum first, then the
 * exponentials and the weighted sum.  No blocking, no online recurrence, no shared code
 * with the CUDA library.  Only tests, the smoke check and the benchmark's CPU-baseline
 * leg may call this.
 *
 * bf16 inputs are widened exactly (bit pattern << 16 is the fp32 with the same value).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int wmtp_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * q    : [Hq][D] bf16 bits
 * K, V : [Hkv][rows][D] bf16 bits, consecutive KV heads `head_stride` elements apart
 * keys : n row indices (the key set, any order), or NULL for rows 0..n-1
 * Query head h reads KV head h / (Hq/Hkv).
 * out  : [Hq][D] fp64, lse : [Hq] fp64 (natural log).  Heads outside [head_lo, head_hi)
 *        are left untouched.  An empty key set gives out = 0 and lse = -inf.
 * Returns 0, or -1 on a bad argument / failed allocation.
 */
int wmtp_oracle_attention(const uint16_t* q, const uint16_t* K, const uint16_t* V,
                          int64_t head_stride, const int64_t* keys, int64_t n,
                          int Hq, int Hkv, int D, double sm_scale,
                          double* out, double* lse, int head_lo, int head_hi) {
    if (!q || !out || !lse || Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0 || n < 0) return -1;
    if (n > 0 && (!K || !V)) return -1;
    if (head_lo < 0) head_lo = 0;
    if (head_hi > Hq) head_hi = Hq;
    const int G = Hq / Hkv;
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int h = head_lo; h < head_hi; ++h) {
        const int g = h / G;
        const uint16_t* Kg = K + (int64_t)g * head_stride;
        const uint16_t* Vg = V + (int64_t)g * head_stride;
        double* o = out + (int64_t)h * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        if (n == 0) { lse[h] = -INFINITY; continue; }
        double* z = (double*)malloc((size_t)n * sizeof(double));
        double* qd = (double*)malloc((size_t)D * sizeof(double));
        if (!z || !qd) { free(z); free(qd); fail = 1; continue; }
        for (int d = 0; d < D; ++d) qd[d] = bf16_to_f64(q[(int64_t)h * D + d]);
        /* pass 1: z_j = sm_scale * <q, k_j>, m = max_j z_j */
        double m = -INFINITY;
        for (int64_t j = 0; j < n; ++j) {
            const int64_t row = keys ? keys[j] : j;
            const uint16_t* k = Kg + row * D;
            double acc = 0.0;
            for (int d = 0; d < D; ++d) acc += qd[d] * bf16_to_f64(k[d]);
            z[j] = sm_scale * acc;
            if (z[j] > m) m = z[j];
        }
        /* pass 2: Z = sum_j exp(z_j - m), o = sum_j exp(z_j - m) v_j / Z */
        double Z = 0.0;
        for (int64_t j = 0; j < n; ++j) {
            const int64_t row = keys ? keys[j] : j;
            const uint16_t* v = Vg + row * D;
            const double p = exp(z[j] - m);
            Z += p;
            for (int d = 0; d < D; ++d) o[d] += p * bf16_to_f64(v[d]);
        }
        for (int d = 0; d < D; ++d) o[d] /= Z;
        lse[h] = m + log(Z);
        free(z);
        free(qd);
    }
    return fail ? -1 : 0;
}

/*
 * fp8 KV variant (Section 6, "Robustness to KV-cache quantization": the KV dtype only sets the bytes
 * per entry; the key set and the attention are unchanged).  K and V hold e4m3 codes -- 1 sign, 4
 * exponent (bias 7), 3 mantissa bits; exponent 0 is subnormal (m/8 * 2^-6); exponent 15 with
 * mantissa 7 is NaN, there are no infinities, the largest finite value is 448 -- and the value of
 * an entry of KV head g is code_value * k_scale[g] (resp. v_scale[g]).
 */
static double e4m3_to_f64(uint8_t b) {
    const int s = b >> 7, e = (b >> 3) & 15, m = b & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return s ? -v : v;
}

/* Same contract as wmtp_oracle_attention, with K, V : [Hkv][rows][D] e4m3 codes (head_stride in
 * elements) and per-KV-head dequantisation scales k_scale, v_scale : [Hkv] fp32. */
int wmtp_oracle_attention_f8(const uint16_t* q, const uint8_t* K, const uint8_t* V,
                             int64_t head_stride, const int64_t* keys, int64_t n,
                             int Hq, int Hkv, int D, double sm_scale,
                             const float* k_scale, const float* v_scale,
                             double* out, double* lse, int head_lo, int head_hi) {
    if (!q || !out || !lse || !k_scale || !v_scale || Hq <= 0 || Hkv <= 0 || D <= 0 || Hq % Hkv != 0 || n < 0) return -1;
    if (n > 0 && (!K || !V)) return -1;
    if (head_lo < 0) head_lo = 0;
    if (head_hi > Hq) head_hi = Hq;
    const int G = Hq / Hkv;
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int h = head_lo; h < head_hi; ++h) {
        const int g = h / G;
        const uint8_t* Kg = K + (int64_t)g * head_stride;
        const uint8_t* Vg = V + (int64_t)g * head_stride;
        const double ks = (double)k_scale[g], vs = (double)v_scale[g];
        double* o = out + (int64_t)h * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        if (n == 0) { lse[h] = -INFINITY; continue; }
        double* z = (double*)malloc((size_t)n * sizeof(double));
        double* qd = (double*)malloc((size_t)D * sizeof(double));
        if (!z || !qd) { free(z); free(qd); fail = 1; continue; }
        for (int d = 0; d < D; ++d) qd[d] = bf16_to_f64(q[(int64_t)h * D + d]);
        double m = -INFINITY;
        for (int64_t j = 0; j < n; ++j) {
            const int64_t row = keys ? keys[j] : j;
            const uint8_t* k = Kg + row * D;
            double acc = 0.0;
            for (int d = 0; d < D; ++d) acc += qd[d] * (e4m3_to_f64(k[d]) * ks);
            z[j] = sm_scale * acc;
            if (z[j] > m) m = z[j];
        }
        double Z = 0.0;
        for (int64_t j = 0; j < n; ++j) {
            const int64_t row = keys ? keys[j] : j;
            const uint8_t* v = Vg + row * D;
            const double p = exp(z[j] - m);
            Z += p;
            for (int d = 0; d < D; ++d) o[d] += p * (e4m3_to_f64(v[d]) * vs);
        }
        for (int d = 0; d < D; ++d) o[d] /= Z;
        lse[h] = m + log(Z);
        free(z);
        free(qd);
    }
    return fail ? -1 : 0;
}
