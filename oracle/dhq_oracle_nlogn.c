/*
 * Second CPU baseline for the DHQ forward pass (arXiv 2508.13478): one quantized layer with the
 * rotation of Eq. 3 computed as an O(n log n) in-place butterfly instead of the O(n^2)
 * entry-by-entry product of the definition.
 *
 * TEST INFRASTRUCTURE ONLY.  This file exists so that the timed CPU baseline is not flattered
 * by the definition's quadratic rotation; it is not the parity reference (dhq_oracle.c is) and
 * the product never calls it.  tests/test_oracle_tiers.py pins it bit-identical to the
 * definition on rotated values, scales, codes, accumulators and outputs.
 *
 * Why the butterfly gives the same bits: output j of the definition is the balanced pairwise
 * fp32 sum, in index order, of the signed inputs; stage h of the butterfly (pairs (i, i+h) with
 * (i & h) == 0 become (a+b, a-b), h = 1, 2, 4, ...) forms exactly the partial sums of that tree
 * one level at a time, each with one fp32 rounding.
 * Everything after the rotation follows Section III-B/C step by step as in the definition:
 * absmax (per token or frozen), s = a/qmax and inv = qmax/a in fp32, round-half-even codes,
 * exact integer product, fp64 dequantization, bias and sine.
 * Build with -O2 -ffp-contract=off -fno-fast-math.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_API __attribute__((visibility("default")))

static void butterfly_f32(float *o, int n)
{
    for (int h = 1; h < n; h *= 2)
        for (int i = 0; i < n; i += 2 * h)
            for (int j = i; j < i + h; ++j) {
                float a = o[j], b = o[j + h];
                o[j] = a + b;
                o[j + h] = a - b;
            }
}

/* Same arguments and outputs as the definition's layer routine; rotate is 0 or 1 (the
 * two-sided transform is not offered here).  Returns 0, -3 on an accumulator outside int32,
 * -4 for rotate == 2. */
ORC_API int dhq_orcn_layer(const float *X, int64_t n, int K_pad, int M_pad, const int32_t *qw,
                           const float *s_w, const float *b_pad, int a_bits, int per_token,
                           float a_frozen, int apply_sine, double omega0, int rotate, float *Xrot,
                           int32_t *codes, float *s_x, int64_t *acc, double *Y)
{
    if (rotate != 0 && rotate != 1) return -4;
    const float qmaxf = (float)((1 << (a_bits - 1)) - 1);
    const int32_t qmax = (1 << (a_bits - 1)) - 1;
    int overflow = 0;
#pragma omp parallel
    {
        float *xr = (float *)malloc(sizeof(float) * (size_t)K_pad);
        int32_t *q = (int32_t *)malloc(sizeof(int32_t) * (size_t)K_pad);
#pragma omp for schedule(static)
        for (int64_t t = 0; t < n; ++t) {
            memcpy(xr, X + t * K_pad, sizeof(float) * (size_t)K_pad);
            if (rotate) butterfly_f32(xr, K_pad);
            float a = a_frozen;
            if (per_token) {
                a = 0.0f;
                for (int k = 0; k < K_pad; ++k) {
                    float v = fabsf(xr[k]);
                    if (v > a) a = v;
                }
            }
            float s = 0.0f, inv = 0.0f;
            if (a > 0.0f && !isinf(qmaxf / a)) { /* no finite scale: treated like a = 0 */
                s = a / qmaxf;
                inv = qmaxf / a;
            }
            for (int k = 0; k < K_pad; ++k) {
                float r = rintf(xr[k] * inv);
                if (r > (float)qmax) r = (float)qmax;
                if (r < (float)-qmax) r = (float)-qmax;
                q[k] = (int32_t)r;
            }
            if (Xrot) memcpy(Xrot + t * K_pad, xr, sizeof(float) * (size_t)K_pad);
            if (codes) memcpy(codes + t * K_pad, q, sizeof(int32_t) * (size_t)K_pad);
            if (s_x) s_x[t] = s;
            for (int m = 0; m < M_pad; ++m) {
                const int32_t *wr = qw + (size_t)m * K_pad;
                int64_t sum = 0;
                for (int k = 0; k < K_pad; ++k) sum += (int64_t)q[k] * (int64_t)wr[k];
                if (sum > INT32_MAX || sum < INT32_MIN) {
#pragma omp atomic write
                    overflow = 1;
                }
                if (acc) acc[t * M_pad + m] = sum;
                if (Y) {
                    double z = (double)s_w[m] * (double)s * (double)sum + (double)b_pad[m];
                    Y[t * M_pad + m] = apply_sine ? sin(omega0 * z) : z;
                }
            }
        }
        free(xr);
        free(q);
    }
    return overflow ? -3 : 0;
}
