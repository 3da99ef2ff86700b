// Weight side of DHQ (Eq. 4-5 of the paper, the factor acting on the input dimension, and the
// quantizer of Section III-B), run once per network on the device:
//   pad -> rotate each row by H_K (fp32 butterfly, strides 1, 2, ..., K/2) -> scale by 1/K
//   -> absmax per tensor or per row -> quantize -> write the codes in three layouts.
#include "dhq_internal.cuh"

namespace dhq {

// One block per padded output row; K/2 threads, one butterfly pair each per stage.
__global__ void prep_rotate_kernel(PrepArgs a)
{
    extern __shared__ float row[];
    const int m = blockIdx.x, K = a.K;
    for (int k = threadIdx.x; k < K; k += blockDim.x)
        row[k] = (m < a.d_out && k < a.d_in) ? a.W[(size_t)m * a.d_in + k] : 0.0f;
    // phase bound of this row: sum_k |W_mk| + |b_m| (inputs of hidden layers lie in [-1, 1])
    __shared__ float red[32];
    float part = 0.f;
    __syncthreads();
    for (int k = threadIdx.x; k < K; k += blockDim.x) part += fabsf(row[k]);
    for (int o = 16; o; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = part;
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.f;
        for (int i = 0; i < (blockDim.x + 31) / 32; ++i) s += red[i];
        float bm = (m < a.d_out) ? fabsf(a.b[m]) : 0.f;
        a.dev.row_l1[m] = s + bm; // |W_m . x + b_m| <= this for inputs in [-1, 1]
        a.dev.bias[m] = (m < a.d_out) ? a.b[m] : 0.0f;
    }
    for (int h = 1; h < (a.rotate ? K : 1); h <<= 1) {
        __syncthreads();
        for (int p = threadIdx.x; p < K / 2; p += blockDim.x) {
            int i = ((p & ~(h - 1)) << 1) | (p & (h - 1));
            float x = row[i], y = row[i + h];
            row[i] = __fadd_rn(x, y);
            row[i + h] = __fsub_rn(x, y);
        }
    }
    __syncthreads();
    const float invK = a.rotate ? 1.0f / (float)K : 1.0f; // power of two: exact
    float amax = 0.f;
    for (int k = threadIdx.x; k < K; k += blockDim.x) {
        float v = __fmul_rn(row[k], invK);
        a.dev.w_rot[(size_t)m * K + k] = v;
        amax = fmaxf(amax, fabsf(v));
    }
    for (int o = 16; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
    __syncthreads();
    if (threadIdx.x == 0) {
        float r = 0.f;
        for (int i = 0; i < (blockDim.x + 31) / 32; ++i) r = fmaxf(r, red[i]);
        a.dev.row_absmax[m] = r;
    }
}

// DHQ_ROT_BOTH, output-side factor of Eq. 4: one block per column k; the column of the row-rotated
// weights goes through the same fp32 butterfly over the M rows and is scaled by the exact 1/M.
__global__ void prep_rotate_cols_kernel(PrepArgs a)
{
    extern __shared__ float col[];
    const int k = blockIdx.x, K = a.K, M = a.M;
    for (int m = threadIdx.x; m < M; m += blockDim.x) col[m] = a.dev.w_rot[(size_t)m * K + k];
    for (int h = 1; h < M; h <<= 1) {
        __syncthreads();
        for (int p = threadIdx.x; p < M / 2; p += blockDim.x) {
            int i = ((p & ~(h - 1)) << 1) | (p & (h - 1));
            float x = col[i], y = col[i + h];
            col[i] = __fadd_rn(x, y);
            col[i + h] = __fsub_rn(x, y);
        }
    }
    __syncthreads();
    const float invM = 1.0f / (float)M; // power of two: exact
    for (int m = threadIdx.x; m < M; m += blockDim.x) a.dev.w_rot[(size_t)m * K + k] = __fmul_rn(col[m], invM);
}

// Row absmax of the final rotated weights (after the column pass).
__global__ void prep_row_absmax_kernel(PrepArgs a)
{
    __shared__ float red[32];
    const int m = blockIdx.x, K = a.K;
    float amax = 0.f;
    for (int k = threadIdx.x; k < K; k += blockDim.x) amax = fmaxf(amax, fabsf(a.dev.w_rot[(size_t)m * K + k]));
    for (int o = 16; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
    __syncthreads();
    if (threadIdx.x == 0) {
        float r = 0.f;
        for (int i = 0; i < (blockDim.x + 31) / 32; ++i) r = fmaxf(r, red[i]);
        a.dev.row_absmax[m] = r;
    }
}

// One block: per-tensor or per-row scales.
__global__ void prep_scales_kernel(PrepArgs a)
{
    __shared__ float tensor_max;
    if (threadIdx.x == 0) {
        float r = 0.f;
        for (int m = 0; m < a.M; ++m) r = fmaxf(r, a.dev.row_absmax[m]);
        tensor_max = r;
    }
    __syncthreads();
    const float qmaxf = qmax_of(a.bits);
    for (int m = threadIdx.x; m < a.M; m += blockDim.x) {
        float s, inv;
        scales_of(a.per_channel ? a.dev.row_absmax[m] : tensor_max, qmaxf, s, inv);
        a.dev.s_w[m] = s;
        a.dev.inv_w[m] = inv;
    }
}

__global__ void prep_quant_kernel(PrepArgs a)
{
    const int K = a.K, M = a.M, Mt = a.Mt;
    const float qmaxf = qmax_of(a.bits);
    const int total = Mt * K;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        int m = idx / K, k = idx % K;
        int q = 0;
        if (m < M) q = quantize(a.dev.w_rot[(size_t)m * K + k], a.dev.inv_w[m], qmaxf);
        if (m < M) {
            a.dev.qw[(size_t)m * K + k] = (int8_t)q;
            ((int8_t *)a.dev.qw_k4m)[((size_t)(k >> 2) * M + m) * 4 + (k & 3)] = (int8_t)q;
        }
        const int row = a.permute_rows ? fused_column(m, M) : m;
        a.dev.qw_umma[umma_offset(row, k, Mt, a.dev.slab_k)] = (uint8_t)(int8_t)q;
    }
}

// Bound of the phase omega0 (s_w s_x acc + b) that the epilogue of a hidden layer sees, over all
// inputs in [-1, 1]^K whose codes do not saturate: the unquantized bound sum_k |W_mk| + |b_m|
// plus what the two quantizers can add.  With s_x q_x = x~ + e_x, |e_x| <= s_x / 2 and
// s_w q_w = w~ + e_w, |e_w| <= s_w / 2:
//   s_w s_x acc = W x + sum_k e_w x~_k + sum_k s_w q_w e_x
//   |sum e_w x~|    <= (s_w / 2) * sum_k |x~_k|,  sum |x~_k| <= K sqrt(K) rotated (||x~||_2 = sqrt(K) ||x||_2), K unrotated
//   |sum s_w q_w e_x| <= (s_x / 2) * s_w * sum_k |q_w[m][k]|,  s_x <= max |x~| / qmax <= K / qmax rotated, 1 / qmax unrotated.
// The maximum over the rows goes to a.phase_bound; it decides between the fast and the wide sine.
__global__ void prep_bound_kernel(PrepArgs a)
{
    __shared__ float red[32];
    const int K = a.K;
    const float xsum = a.rotate ? (float)K * sqrtf((float)K) : (float)K;
    const float sx_max = (a.rotate ? (float)K : 1.0f) / qmax_of(a.a_bits);
    float worst = 0.f;
    for (int m = threadIdx.x; m < a.M; m += blockDim.x) {
        float qsum = 0.f;
        for (int k = 0; k < K; ++k) qsum += fabsf((float)a.dev.qw[(size_t)m * K + k]);
        atomicAdd(a.code_l1, (unsigned long long)qsum); // exact: at most 512 * 127 per row
        const float sw = a.dev.s_w[m];
        const float slack = 0.5f * sw * xsum + 0.5f * sx_max * sw * qsum;
        worst = fmaxf(worst, (float)a.omega0 * (a.dev.row_l1[m] + slack) * 1.0001f);
    }
    for (int o = 16; o; o >>= 1) worst = fmaxf(worst, __shfl_xor_sync(0xffffffffu, worst, o));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = worst;
    __syncthreads();
    if (threadIdx.x == 0) {
        float r = 0.f;
        for (int i = 0; i < (blockDim.x + 31) / 32; ++i) r = fmaxf(r, red[i]);
        *a.phase_bound = r;
    }
}

// Two-sided transform, layer 1 (K = 4): the rotated padded coordinate has the codes [qs, qd, qs, qd],
// so acc_m = qs u_m + qd v_m with u_m = q[m][0] + q[m][2], v_m = q[m][1] + q[m][3], and the rotated
// accumulators are acc'_j = qs (H_M u)_j + qd (H_M v)_j.  One block computes H_M u and H_M v.
__global__ void prep_l1_both_kernel(LayerDev dev)
{
    extern __shared__ int uv[]; // [2][M]
    const int M = dev.M;
    for (int m = threadIdx.x; m < M; m += blockDim.x) {
        const int8_t *q = dev.qw + (size_t)m * 4;
        uv[m] = (int)q[0] + (int)q[2];
        uv[M + m] = (int)q[1] + (int)q[3];
    }
    for (int h = 1; h < M; h <<= 1) {
        __syncthreads();
        for (int p = threadIdx.x; p < M; p += blockDim.x) { // M/2 pairs for each of the two vectors
            const int which = p / (M / 2), j = p % (M / 2);
            const int i = which * M + (((j & ~(h - 1)) << 1) | (j & (h - 1)));
            const int x = uv[i], y = uv[i + h];
            uv[i] = x + y;
            uv[i + h] = x - y;
        }
    }
    __syncthreads();
    for (int m = threadIdx.x; m < M; m += blockDim.x) {
        dev.l1U[m] = uv[m];
        dev.l1V[m] = uv[M + m];
    }
}

// Epilogue constants in fp64, rounded once: cA = fl32(A), cA_lo = fl32(A - cA) with
// A = f * s_w[m] (* s_x when the activation scale is per tensor), cB = fl32(f * b[m]),
// f = omega0 for sine layers and 1 for the last layer.  Also derives s_x and inv from the frozen
// absmax in per-tensor mode.
__global__ void finalize_kernel(LayerDev dev, int a_bits, int per_token, int sine, double omega0)
{
    __shared__ float s_x_sh;
    if (threadIdx.x == 0) {
        float s = 1.0f;
        if (!per_token) {
            float inv;
            scales_of(dev.act[0], qmax_of(a_bits), s, inv);
            dev.act[1] = s;
            dev.act[2] = inv;
        }
        s_x_sh = s;
    }
    __syncthreads();
    const double f = sine ? omega0 : 1.0;
    for (int m = threadIdx.x; m < dev.M; m += blockDim.x) {
        double A = f * (double)dev.s_w[m] * (per_token ? 1.0 : (double)s_x_sh);
        float hi = (float)A;
        dev.cA[m] = hi;
        dev.cA_lo[m] = (float)(A - (double)hi);
        dev.cB[m] = (float)(f * (double)dev.bias[m]);
        if (dev.epi_mode == EPI_SINE_FIXED) {
            const double inv_two_pi = 0.15915494309189533576888;
            const int8_t *q = dev.qw + (size_t)m * 4;   // layer 1: K = 4
            double u = (double)((int)q[0] + (int)q[2]), v = (double)((int)q[1] + (int)q[3]);
            if (dev.has_uv) { // two-sided transform: the phase of output j comes from the rotated sums
                u = (double)dev.l1U[m];
                v = (double)dev.l1V[m];
            }
            auto to_fix = [](double turns) { return (uint32_t)(unsigned long long)llrint(turns * 4294967296.0); };
            dev.fxP[m] = to_fix(A * u * inv_two_pi);
            dev.fxQ[m] = to_fix(A * v * inv_two_pi);
            dev.fxB[m] = to_fix(f * (double)dev.bias[m] * inv_two_pi);
        }
    }
}

cudaError_t launch_prepare(const PrepArgs &a, cudaStream_t st, int64_t *launches)
{
    int threads = a.K / 2 < 32 ? 32 : a.K / 2;
    prep_rotate_kernel<<<a.M, threads, a.K * sizeof(float), st>>>(a);
    if (a.rotate == 2) {
        int tc = a.M / 2 < 32 ? 32 : a.M / 2;
        prep_rotate_cols_kernel<<<a.K, tc, a.M * sizeof(float), st>>>(a);
        prep_row_absmax_kernel<<<a.M, 128, 0, st>>>(a);
        *launches += 2;
    }
    prep_scales_kernel<<<1, 256, 0, st>>>(a);
    int total = a.Mt * a.K;
    prep_quant_kernel<<<(total + 255) / 256, 256, 0, st>>>(a);
    prep_bound_kernel<<<1, 256, 0, st>>>(a);
    *launches += 4;
    if (a.dev.has_uv) {
        prep_l1_both_kernel<<<1, 256, 2 * a.M * sizeof(int), st>>>(a.dev);
        *launches += 1;
    }
    return cudaGetLastError();
}

cudaError_t launch_finalize(const LayerDev &dev, int a_bits, int per_token, int sine, double omega0,
                            cudaStream_t st, int64_t *launches)
{
    finalize_kernel<<<1, 256, 0, st>>>(dev, a_bits, per_token, sine, omega0);
    *launches += 1;
    return cudaGetLastError();
}

} // namespace dhq
