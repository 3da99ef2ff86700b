/*
 * CPU oracle for the DHQ quantized INR forward pass (arXiv 2508.13478).
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, definition-shaped implementation used to
 * check the CUDA library and to time a CPU baseline.  It shares no code with the CUDA path and
 * the product never calls it.
 *
 * What the paper fixes and what it leaves open:
 *   - Eq. 3 (Section III-B) defines the Hadamard matrix by the Sylvester recursion; the matrix
 *     is built here literally that way and every rotation multiplies by it entry by entry.
 *   - Eq. 4-5 rotate a weight matrix; the inference path uses the input-side factor W H_K / K
 *     (so that W x = (W H_K / K)(H_K x), H being symmetric), activations are rotated
 *     un-normalised, and the exact power-of-two 1/K lives in the weights.
 *   - The "standard quantizer" (Section III-B) is read as symmetric absmax, qmax = 2^(b-1)-1,
 *     s = a/qmax and inv = qmax/a both as IEEE fp32 divisions, q = clamp(rint(fl32(v*inv))) with
 *     round-half-to-even, a = 0 giving s = inv = 0.
 *   - The output layer has no activation (Section III-C); hidden layers apply sin(omega0 * z).
 *   - Section IV also evaluates WIRE, "featuring wavelet activation functions", without giving the
 *     function.  Reading (gabor_s0 > 0): the real-valued Gabor wavelet of the WIRE paper,
 *     psi(z) = sin(omega0 z) * exp(-(s0 z)^2); its complex form exp(j omega0 z - |s0 z|^2) is not
 *     built.  gabor_s0 = 0 is the sine.
 *   - rotate = 2 is the two-sided transform of Eq. 4-5 taken literally: W~ = H_M W H_K / (K M)
 *     (rows rotated first, then columns, both as pinned fp32 pairwise sums, both scales exact
 *     powers of two), and since H_M H_M = M I the layer output is z = H_M d + b with
 *     d_m = s_w[m] s_x acc_m.  That second rotation decides no integer, so it is an explicit
 *     fp64 matrix product.
 *
 * Parity pins (tests/test_oracle_*.py): Hadamard recursion vs closed form and H H^T = nI;
 * rotation vs an exact integer product and vs fp64; W x = (W H/K)(H x); Frobenius norm
 * preservation; quantizer error <= s/2; brute force on 4-wide layers; convergence of the whole
 * network to the unquantized fp64 SIREN as the bit-width grows; the per-output-channel branch of
 * the weight quantizer by a hand-derived fixture and row-wise properties; every code of weights
 * and activations against the same layer stated in fp64 with the orthonormal scaling (they may
 * differ by one step only where the value to be rounded is within 1e-4 of a half-integer).
 * Parity unpinned by the paper: the order of the fp32 additions inside a rotation (pinned here
 * as a balanced pairwise sum in index order) and the rounding mode / granularity of the
 * quantizer (pinned as stated above).
 *
 * Floating point: rotations, absmax, scales and the quantizer multiply are IEEE fp32 (they
 * decide integer codes, so both implementations must take them in the same precision); the
 * integer matmul is exact; the dequantize / bias / sine epilogue is fp64.
 * Build with -O2 -ffp-contract=off -fno-fast-math so that no fp32 step is fused or reordered.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_API __attribute__((visibility("default")))

ORC_API int dhq_orc_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Eq. 3: H_1 = [1], H_2n = [[H_n, H_n], [H_n, -H_n]].  H is n*n int8, row-major. */
ORC_API int dhq_orc_hadamard(int n, int8_t *H)
{
    if (n < 1 || (n & (n - 1)) != 0) return -1;
    H[0] = 1;
    for (int m = 1; m < n; m *= 2) {
        /* the top-left m*m block holds H_m (with row stride n); fill the other three blocks */
        for (int i = 0; i < m; ++i)
            for (int j = 0; j < m; ++j) {
                int8_t h = H[(size_t)i * n + j];
                H[(size_t)i * n + (j + m)] = h;
                H[(size_t)(i + m) * n + j] = h;
                H[(size_t)(i + m) * n + (j + m)] = (int8_t)(-h);
            }
    }
    return 0;
}

/* Balanced pairwise fp32 sum of t[lo .. lo+len-1] in index order: (left half) + (right half). */
static float pairwise_sum_f32(const float *t, int lo, int len)
{
    if (len == 1) return t[lo];
    float a = pairwise_sum_f32(t, lo, len / 2);
    float b = pairwise_sum_f32(t, lo + len / 2, len / 2);
    return a + b;
}

/* out[j] = sum_l H[j][l] * v[l]  (the vector form below Eq. 3), each product an exact sign
 * flip, the sum taken as a balanced pairwise fp32 sum in index order.  scratch: n floats. */
static void rotate_one(const int8_t *H, int n, const float *v, float *out, float *scratch)
{
    for (int j = 0; j < n; ++j) {
        const int8_t *row = H + (size_t)j * n;
        for (int l = 0; l < n; ++l) scratch[l] = (row[l] > 0) ? v[l] : -v[l];
        out[j] = pairwise_sum_f32(scratch, 0, n);
    }
}

ORC_API void dhq_orc_rotate_rows(const int8_t *H, int n, int64_t rows, const float *V, float *out)
{
#pragma omp parallel
    {
        float *scratch = (float *)malloc(sizeof(float) * (size_t)n);
#pragma omp for schedule(static)
        for (int64_t r = 0; r < rows; ++r)
            rotate_one(H, n, V + r * n, out + r * n, scratch);
        free(scratch);
    }
}

/* The same rotation as an in-place O(n log n) butterfly (strides 1, 2, 4, ...; the pair
 * (i, i+h) becomes (a+b, a-b)).  Not part of the definition: it exists so that the CPU baseline
 * can also be timed without the O(n^2) cost, and the tests check it is bit-identical. */
ORC_API void dhq_orc_rotate_rows_butterfly(int n, int64_t rows, const float *V, float *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        float *o = out + r * n;
        memcpy(o, V + r * n, sizeof(float) * (size_t)n);
        for (int h = 1; h < n; h *= 2)
            for (int i = 0; i < n; ++i)
                if ((i & h) == 0) {
                    float a = o[i], b = o[i + h];
                    o[i] = a + b;
                    o[i + h] = a - b;
                }
    }
}

ORC_API float dhq_orc_absmax(const float *v, int64_t count)
{
    float a = 0.0f;
    for (int64_t i = 0; i < count; ++i) {
        float x = fabsf(v[i]);
        if (x > a) a = x;
    }
    return a;
}

/* Symmetric absmax quantizer scales: s = a/qmax, inv = qmax/a (fp32 divisions); a = 0 -> 0, 0.
 * Reading of the "standard quantizer" (Section III-B) at its degenerate end: an absmax so small
 * that qmax/a overflows fp32 (a below about 3.7e-37 at 8 bits) has no finite scale to round
 * with; it is treated like a = 0 (all codes zero, s = 0). */
ORC_API void dhq_orc_scales(float a, int bits, float *s, float *inv)
{
    float qmax = (float)((1 << (bits - 1)) - 1);
    *s = 0.0f;
    *inv = 0.0f;
    if (a > 0.0f) {
        float i = qmax / a;
        if (!isinf(i)) {
            *s = a / qmax;
            *inv = i;
        }
    }
}

/* q = clamp(round-half-even(fl32(v * inv)), -qmax, +qmax). */
ORC_API void dhq_orc_quantize(const float *v, int64_t count, float inv, int bits, int32_t *q)
{
    int32_t qmax = (1 << (bits - 1)) - 1;
    for (int64_t i = 0; i < count; ++i) {
        float t = v[i] * inv;
        float r = rintf(t); /* default rounding mode: to nearest, ties to even */
        if (r > (float)qmax) r = (float)qmax;
        if (r < (float)-qmax) r = (float)-qmax;
        q[i] = (int32_t)r;
    }
}

/*
 * Weight side (Eq. 4-5, input-side factor): pad W[d_out][d_in] with zeros to [M_pad][K_pad],
 * rotate each row (rotate != 0), scale by the exact 1/K_pad, for rotate = 2 also rotate each column
 * and scale by the exact 1/M_pad, quantize per tensor
 * (per_channel = 0) or per output row.  Outputs: Wrot [M_pad][K_pad] fp32, q [M_pad][K_pad],
 * s_w [M_pad] (per-tensor: the same value repeated).
 */
ORC_API int dhq_orc_prepare_layer(const float *W, int d_out, int d_in, int M_pad, int K_pad,
                                  int bits, int per_channel, int rotate, float *Wrot, int32_t *q,
                                  float *s_w)
{
    if (d_out > M_pad || d_in > K_pad) return -1;
    size_t cnt = (size_t)M_pad * K_pad;
    float *padded = (float *)calloc(cnt, sizeof(float));
    int8_t *H = (int8_t *)malloc((size_t)K_pad * K_pad);
    if (!padded || !H || dhq_orc_hadamard(K_pad, H) != 0) {
        free(padded);
        free(H);
        return -2;
    }
    for (int m = 0; m < d_out; ++m)
        for (int k = 0; k < d_in; ++k) padded[(size_t)m * K_pad + k] = W[(size_t)m * d_in + k];
    if (rotate) {
        dhq_orc_rotate_rows(H, K_pad, M_pad, padded, Wrot);
        float invK = 1.0f / (float)K_pad; /* power of two: exact */
        for (size_t i = 0; i < cnt; ++i) Wrot[i] = Wrot[i] * invK;
    } else {
        memcpy(Wrot, padded, cnt * sizeof(float));
    }
    if (rotate == 2) {
        /* output-side factor of Eq. 4: every column k becomes Tree(H_M column_k) / M */
        int8_t *HM = (int8_t *)malloc((size_t)M_pad * M_pad);
        float *colT = (float *)malloc(cnt * sizeof(float)), *rotT = (float *)malloc(cnt * sizeof(float));
        if (!HM || !colT || !rotT || dhq_orc_hadamard(M_pad, HM) != 0) {
            free(HM); free(colT); free(rotT); free(padded); free(H);
            return -2;
        }
        for (int m = 0; m < M_pad; ++m)
            for (int k = 0; k < K_pad; ++k) colT[(size_t)k * M_pad + m] = Wrot[(size_t)m * K_pad + k];
        dhq_orc_rotate_rows(HM, M_pad, K_pad, colT, rotT);
        float invM = 1.0f / (float)M_pad; /* power of two: exact */
        for (int m = 0; m < M_pad; ++m)
            for (int k = 0; k < K_pad; ++k) Wrot[(size_t)m * K_pad + k] = rotT[(size_t)k * M_pad + m] * invM;
        free(HM); free(colT); free(rotT);
    }
    if (per_channel) {
        for (int m = 0; m < M_pad; ++m) {
            float s, inv;
            dhq_orc_scales(dhq_orc_absmax(Wrot + (size_t)m * K_pad, K_pad), bits, &s, &inv);
            s_w[m] = s;
            dhq_orc_quantize(Wrot + (size_t)m * K_pad, K_pad, inv, bits, q + (size_t)m * K_pad);
        }
    } else {
        float s, inv;
        dhq_orc_scales(dhq_orc_absmax(Wrot, (int64_t)cnt), bits, &s, &inv);
        for (int m = 0; m < M_pad; ++m) s_w[m] = s;
        dhq_orc_quantize(Wrot, (int64_t)cnt, inv, bits, q);
    }
    free(padded);
    free(H);
    return 0;
}

/*
 * Per-token absmax of the rotated layer input: amax[t] = max_j |(H_K X_t)_j|.  Used to freeze a
 * per-tensor activation scale (the maximum of amax over the calibration set).
 */
ORC_API void dhq_orc_rotated_absmax(const float *X, int64_t n, int K_pad, int rotate, float *amax)
{
    int8_t *H = (int8_t *)malloc((size_t)K_pad * K_pad);
    dhq_orc_hadamard(K_pad, H);
#pragma omp parallel
    {
        float *scratch = (float *)malloc(sizeof(float) * (size_t)K_pad);
        float *xr = (float *)malloc(sizeof(float) * (size_t)K_pad);
#pragma omp for schedule(static)
        for (int64_t t = 0; t < n; ++t) {
            if (rotate) rotate_one(H, K_pad, X + t * K_pad, xr, scratch);
            else memcpy(xr, X + t * K_pad, sizeof(float) * (size_t)K_pad);
            amax[t] = dhq_orc_absmax(xr, K_pad);
        }
        free(scratch);
        free(xr);
    }
    free(H);
}

/*
 * One quantized layer for n tokens (Section III-B/C):
 *   x~ = H_K X_t (un-normalised)          -> Xrot  [n][K_pad] fp32
 *   a  = per-token absmax, or a_frozen     -> s_x   [n] fp32 (per-tensor: the same value)
 *   q  = quantize(x~)                      -> codes [n][K_pad]
 *   acc[m] = sum_k q[k] * qw[m][k]         -> acc   [n][M_pad] int64 (exact)
 *   z = s_w[m] * s_x * acc + b[m] in fp64; Y = sin(omega0 z) (times exp(-(gabor_s0 z)^2) if gabor_s0 > 0)
 *       for hidden layers, z for the last
 *                                          -> Y     [n][M_pad] fp64
 *   rotate = 2: z = H_M (s_w s_x acc) + b instead (fp64 matrix product)
 * Any output pointer may be NULL.  Returns 0, or -3 if an accumulator leaves the int32 range.
 */
static double activation(double z, double omega0, double gabor_s0)
{
    double y = sin(omega0 * z);
    if (gabor_s0 > 0.0) y *= exp(-(gabor_s0 * z) * (gabor_s0 * z));
    return y;
}

ORC_API int dhq_orc_layer(const float *X, int64_t n, int K_pad, int M_pad, const int32_t *qw,
                          const float *s_w, const float *b_pad, int a_bits, int per_token,
                          float a_frozen, int apply_sine, double omega0, int rotate, float *Xrot,
                          int32_t *codes, float *s_x, int64_t *acc, double *Y, double gabor_s0)
{
    int8_t *H = (int8_t *)malloc((size_t)K_pad * K_pad);
    int8_t *HM = (int8_t *)malloc((size_t)M_pad * M_pad);
    if (!H || !HM || dhq_orc_hadamard(K_pad, H) != 0 || dhq_orc_hadamard(M_pad, HM) != 0) {
        free(H);
        free(HM);
        return -2;
    }
    int overflow = 0;
#pragma omp parallel
    {
        float *scratch = (float *)malloc(sizeof(float) * (size_t)K_pad);
        float *xr = (float *)malloc(sizeof(float) * (size_t)K_pad);
        int32_t *q = (int32_t *)malloc(sizeof(int32_t) * (size_t)K_pad);
        double *dq = (double *)malloc(sizeof(double) * (size_t)M_pad);
#pragma omp for schedule(static)
        for (int64_t t = 0; t < n; ++t) {
            const float *x = X + t * K_pad;
            if (rotate) rotate_one(H, K_pad, x, xr, scratch);
            else memcpy(xr, x, sizeof(float) * (size_t)K_pad);
            float a = per_token ? dhq_orc_absmax(xr, K_pad) : a_frozen;
            float s, inv;
            dhq_orc_scales(a, a_bits, &s, &inv);
            dhq_orc_quantize(xr, K_pad, inv, a_bits, q);
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
                if (rotate == 2) {
                    dq[m] = (double)s_w[m] * (double)s * (double)sum; /* still in the rotated output basis */
                } else if (Y) {
                    double z = (double)s_w[m] * (double)s * (double)sum + (double)b_pad[m];
                    Y[t * M_pad + m] = apply_sine ? activation(z, omega0, gabor_s0) : z;
                }
            }
            if (rotate == 2 && Y) {
                /* z = H_M d + b: undoes the output-side factor of W~ (H_M H_M = M I, the 1/M is in W~) */
                for (int j = 0; j < M_pad; ++j) {
                    const int8_t *hr = HM + (size_t)j * M_pad;
                    double z = 0.0;
                    for (int m = 0; m < M_pad; ++m) z += (hr[m] > 0) ? dq[m] : -dq[m];
                    z += (double)b_pad[j];
                    Y[t * M_pad + j] = apply_sine ? activation(z, omega0, gabor_s0) : z;
                }
            }
        }
        free(scratch);
        free(xr);
        free(q);
        free(dq);
    }
    free(H);
    free(HM);
    return overflow ? -3 : 0;
}
