// Layer-by-layer path: one kernel pass per layer with activations in device memory between
// layers.  It serves the debug dump (every intermediate of Section III-B/C observable) and the
// per-tensor calibration passes.  Same per-element arithmetic as the fused kernel (dhq_math.cuh).
//
// A block handles TB tokens: the rotation runs as a shared-memory butterfly, the integer matmul
// as dp4a over weights stored four-k-per-word with the output channel as the fast index.
#include "dhq_internal.cuh"

namespace dhq {

constexpr int TB = 16;        // tokens per block
constexpr int LW_THREADS = 256;

__global__ void __launch_bounds__(LW_THREADS) layer_kernel(LayerArgs a)
{
    __shared__ float xs[TB * 512];
    __shared__ __align__(16) int8_t cs[TB * 512];
    __shared__ float s_tok[TB], inv_tok[TB];
    __shared__ float blockmax[LW_THREADS / 32];
    extern __shared__ double dq[];   // DHQ_ROT_BOTH only: [TB][M] dequantized values in the rotated output basis

    const int K = a.K, M = a.M, tid = threadIdx.x;
    const int64_t base = (int64_t)blockIdx.x * TB;
    const float qmaxf = qmax_of(a.a_bits);

    // layer input (zero rows past the end; they are never written back nor counted)
    for (int idx = tid; idx < TB * K; idx += LW_THREADS) {
        int t = idx / K, k = idx % K;
        int64_t tok = base + t;
        float v = 0.f;
        if (tok < a.n) v = a.X ? a.X[tok * K + k] : (k < 2 ? a.coords[tok * 2 + k] : 0.f);
        xs[idx] = v;
        if (a.dX && tok < a.n) a.dX[tok * K + k] = v;
    }
    // rotation: strides 1, 2, ..., K/2; pair (i, i+h) -> (x+y, x-y)
    for (int h = 1; h < (a.rotate ? K : 1); h <<= 1) {
        __syncthreads();
        for (int p = tid; p < TB * (K / 2); p += LW_THREADS) {
            int t = p / (K / 2), j = p % (K / 2);
            int i = t * K + (((j & ~(h - 1)) << 1) | (j & (h - 1)));
            float x = xs[i], y = xs[i + h];
            xs[i] = __fadd_rn(x, y);
            xs[i + h] = __fsub_rn(x, y);
        }
    }
    __syncthreads();
    // per-token absmax of the rotated input: warp w takes tokens w, w+8
    const int warp = tid >> 5, lane = tid & 31;
    float bmax = 0.f;
    for (int t = warp; t < TB; t += LW_THREADS / 32) {
        float m = 0.f;
        for (int k = lane; k < K; k += 32) m = fmaxf(m, fabsf(xs[t * K + k]));
        for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (base + t < a.n) bmax = fmaxf(bmax, m);
        if (lane == 0) {
            float s, inv;
            if (a.per_token) scales_of(m, qmaxf, s, inv);
            else { s = a.act[1]; inv = a.act[2]; }
            s_tok[t] = s;
            inv_tok[t] = inv;
            if (a.ds_x && base + t < a.n) a.ds_x[base + t] = s;
        }
    }
    if (a.calib_only) {
        if (lane == 0) blockmax[warp] = bmax;
        __syncthreads();
        if (tid == 0) {
            float m = 0.f;
            for (int i = 0; i < LW_THREADS / 32; ++i) m = fmaxf(m, blockmax[i]);
            atomicMax((unsigned int *)a.act, __float_as_uint(m)); // non-negative floats order as uints
        }
        return;
    }
    __syncthreads();
    for (int idx = tid; idx < TB * K; idx += LW_THREADS) {
        int t = idx / K;
        int q = quantize(xs[idx], inv_tok[t], qmaxf);
        cs[idx] = (int8_t)q;
        int64_t tok = base + t;
        if (a.dcodes && tok < a.n) a.dcodes[tok * K + (idx % K)] = (int8_t)q;
    }
    __syncthreads();
    // integer matmul + epilogue: thread -> output channel m, all TB tokens
    const int K4 = K / 4;
    for (int m = tid; m < M; m += LW_THREADS) {
        int acc[TB];
#pragma unroll
        for (int t = 0; t < TB; ++t) acc[t] = 0;
        for (int k4 = 0; k4 < K4; ++k4) {
            int w = (int)a.qw_k4m[(size_t)k4 * M + m];
#pragma unroll
            for (int t = 0; t < TB; ++t)
                acc[t] = __dp4a(((const int *)cs)[t * K4 + k4], w, acc[t]);
        }
        if (a.rotate == 2) {
            // two-sided transform: keep d = s_w s_x acc of every token; the output follows below
            const double sw = (double)a.s_w[m];
#pragma unroll
            for (int t = 0; t < TB; ++t) {
                dq[t * M + m] = sw * (double)s_tok[t] * (double)acc[t];
                int64_t tok = base + t;
                if (a.dacc && tok < a.n) a.dacc[tok * M + m] = acc[t];
            }
            continue;
        }
        const float cA = a.cA[m], cAl = a.cA_lo[m], cB = a.cB[m];
#pragma unroll
        for (int t = 0; t < TB; ++t) {
            int64_t tok = base + t;
            if (tok >= a.n) continue;
            float c_hi = cA, c_lo = cAl;
            if (a.per_token) token_const(cA, cAl, s_tok[t], c_hi, c_lo);
            float y;
            if (a.epi_mode == EPI_SINE_FIXED)
                y = sine_fixed((int)cs[t * K + 0], (int)cs[t * K + 1], a.fxP[m], a.fxQ[m], a.fxB[m]);
            else if (a.gabor_s0 > 0.0 && a.sine)
                y = gabor_epilogue((float)acc[t], c_hi, c_lo, cB, (float)(a.gabor_s0 / a.omega0));
            else if (a.epi_mode == EPI_SINE_MIXED)
                y = epilogue_mixed((float)acc[t], c_hi, c_lo, cB, a.per_token ? kFastPhaseLimitPerToken : kFastPhaseLimit);
            else
                y = epilogue(a.epi_mode, (float)acc[t], c_hi, c_lo, cB);
            if (a.dacc) a.dacc[tok * M + m] = acc[t];
            if (a.Y) a.Y[tok * M + m] = y;
            if (a.out && m < a.d_L) a.out[tok * a.d_L + m] = y;
        }
    }
    if (a.rotate != 2) return;
    // z = H_M d + b (H_M H_M = M I, and the 1/M is in the weights): fp64 butterfly over the M outputs.
    // The sum of up to 512 terms reaches phases of tens of radians that must stay within 1e-5 of
    // the fp64 definition; an fp32 butterfly does not (about 1e-7 rms per radian of phase).
    for (int h = 1; h < M; h <<= 1) {
        __syncthreads();
        for (int p = tid; p < TB * (M / 2); p += LW_THREADS) {
            int t = p / (M / 2), j = p % (M / 2);
            int i = t * M + (((j & ~(h - 1)) << 1) | (j & (h - 1)));
            double x = dq[i], y = dq[i + h];
            dq[i] = x + y;
            dq[i + h] = x - y;
        }
    }
    __syncthreads();
    for (int idx = tid; idx < TB * M; idx += LW_THREADS) {
        int t = idx / M, j = idx % M;
        int64_t tok = base + t;
        if (tok >= a.n) continue;
        double z = dq[idx] + (double)a.bias[j];
        float y;
        if (a.sine) {
            // phase reduced to [-pi, pi] in fp64, then the hardware sine on an fp32 argument
            const double two_pi = 6.283185307179586476925287;
            double ph = a.omega0 * z;
            ph -= two_pi * rint(ph * (1.0 / two_pi));
            y = sin_approx((float)ph);
            if (a.gabor_s0 > 0.0) y = __fmul_rn(y, (float)exp(-(a.gabor_s0 * z) * (a.gabor_s0 * z)));
        } else {
            y = (float)z;
        }
        if (a.Y) a.Y[tok * M + j] = y;
        if (a.out && j < a.d_L) a.out[tok * a.d_L + j] = y;
    }
}

cudaError_t launch_layer(const LayerArgs &a, cudaStream_t st)
{
    if (a.n <= 0) return cudaSuccess;
    int64_t blocks = (a.n + TB - 1) / TB;
    size_t dyn = 0;
    if (a.rotate == 2 && !a.calib_only) {
        dyn = (size_t)TB * a.M * sizeof(double); // up to 64 KB beside the 41 KB of static shared memory
        cudaError_t e = cudaFuncSetAttribute(layer_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TB * 512 * (int)sizeof(double));
        if (e != cudaSuccess) return e;
    }
    layer_kernel<<<(unsigned)blocks, LW_THREADS, dyn, st>>>(a);
    return cudaGetLastError();
}

} // namespace dhq
