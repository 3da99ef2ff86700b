// The two comparison datapaths of the paper's hardware table (Table 2) and motivation figure
// (Section I): W8A32 - weights folded and quantized exactly as for DHQ, activations kept in fp32 -
// and W32A32 - the plain fp32 sinusoidal network.  One kernel pass per layer, activations in device
// memory between layers, fp32 multiply-adds on the CUDA cores.  These exist so that the three
// datapaths can be compared on the same GPU; they are not the product's hot path and not tuned.
//
//   W8A32:  x~ = H_K x (fp32 butterfly, or x itself without the rotation)
//           z  = s_w[m] * sum_k q_w[m][k] x~_k + b[m]          (q_w exact in fp32)
//   W32A32: z  = sum_k W[m][k] x_k + b[m]
//   y = sin(omega0 z) for hidden layers (explicit 2 pi reduction), z for the last layer.
#include <type_traits>
#include "dhq_internal.cuh"

namespace dhq {

constexpr int FTB = 16; // tokens per block
constexpr int FL_THREADS = 256;

__global__ void __launch_bounds__(FL_THREADS) float_layer_kernel(FloatLayerArgs a)
{
    __shared__ __align__(16) float xs[FTB * 512];
    const int K = a.K, M = a.M, tid = threadIdx.x;
    const int64_t base = (int64_t)blockIdx.x * FTB;
    for (int idx = tid; idx < FTB * K; idx += FL_THREADS) {
        const int t = idx / K, k = idx % K;
        const int64_t tok = base + t;
        float v = 0.f;
        if (tok < a.n) v = a.X ? a.X[tok * K + k] : (k < 2 ? a.coords[tok * 2 + k] : 0.f);
        xs[idx] = v;
        if (a.dX && tok < a.n) a.dX[tok * K + k] = v;
    }
    // rotation (W8A32 with the Hadamard fold): strides 1, 2, ..., K/2; pair (i, i+h) -> (x+y, x-y)
    for (int h = 1; h < (a.rotate ? K : 1); h <<= 1) {
        __syncthreads();
        for (int p = tid; p < FTB * (K / 2); p += FL_THREADS) {
            const int t = p / (K / 2), j = p % (K / 2);
            const int i = t * K + (((j & ~(h - 1)) << 1) | (j & (h - 1)));
            const float x = xs[i], y = xs[i + h];
            xs[i] = __fadd_rn(x, y);
            xs[i + h] = __fsub_rn(x, y);
        }
    }
    __syncthreads();
    const int K4 = K / 4;
    // Each thread takes CPT output channels (m, m + FL_THREADS, ...) for all FTB tokens at once, so that one
    // broadcast read of four activations feeds 4 * CPT multiply-adds (with one channel per pass the
    // shared-memory reads, not the FMAs, set the pace).
    auto run = [&](auto cpt_tag) {
        constexpr int CPT = decltype(cpt_tag)::value;
        for (int m0 = tid; m0 < M; m0 += FL_THREADS * CPT) {
            float acc[CPT][FTB];
#pragma unroll
            for (int c = 0; c < CPT; ++c)
#pragma unroll
                for (int t = 0; t < FTB; ++t) acc[c][t] = 0.f;
            for (int k4 = 0; k4 < K4; ++k4) {
                float w[CPT][4];
#pragma unroll
                for (int c = 0; c < CPT; ++c) {
                    const int m = m0 + c * FL_THREADS;
                    if (m < M) {
                        if (a.w8) {
                            const uint32_t word = a.qw_k4m[(size_t)k4 * M + m]; // four consecutive-k codes of channel m
                            w[c][0] = (float)(int8_t)(word & 0xff);
                            w[c][1] = (float)(int8_t)((word >> 8) & 0xff);
                            w[c][2] = (float)(int8_t)((word >> 16) & 0xff);
                            w[c][3] = (float)(int8_t)(word >> 24);
                        } else {
                            const float4 wv = a.w_f32[(size_t)k4 * M + m];
                            w[c][0] = wv.x; w[c][1] = wv.y; w[c][2] = wv.z; w[c][3] = wv.w;
                        }
                    } else {
                        w[c][0] = w[c][1] = w[c][2] = w[c][3] = 0.f;
                    }
                }
#pragma unroll
                for (int t = 0; t < FTB; ++t) {
                    const float4 x = *reinterpret_cast<const float4 *>(&xs[t * K + 4 * k4]);
#pragma unroll
                    for (int c = 0; c < CPT; ++c)
                        acc[c][t] = __fmaf_rn(w[c][3], x.w, __fmaf_rn(w[c][2], x.z, __fmaf_rn(w[c][1], x.y, __fmaf_rn(w[c][0], x.x, acc[c][t]))));
                }
            }
#pragma unroll
            for (int c = 0; c < CPT; ++c) {
                const int m = m0 + c * FL_THREADS;
                if (m >= M) continue;
                const float bm = a.bias[m], sw = a.w8 ? a.s_w[m] : 1.0f;
#pragma unroll
                for (int t = 0; t < FTB; ++t) {
                    const int64_t tok = base + t;
                    if (tok >= a.n) continue;
                    const float z = a.w8 ? __fmaf_rn(acc[c][t], sw, bm) : __fadd_rn(acc[c][t], bm);
                    const float y = a.sine ? sin_wide(__fmul_rn(a.omega0, z)) : z;
                    if (a.Y) a.Y[tok * M + m] = y;
                    if (a.out && m < a.d_L) a.out[tok * a.d_L + m] = y;
                }
            }
        }
    };
    if (M >= 2 * FL_THREADS) run(std::integral_constant<int, 2>());
    else run(std::integral_constant<int, 1>());
}

// fp32 weights of one layer, zero padded to [M][K], as [K/4][M] float4 (four consecutive k of a
// channel per element, the channel as the fast index).
__global__ void prep_float_weights_kernel(const float *W, int d_out, int d_in, int K, int M, float4 *dst)
{
    const int total = (K / 4) * M;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
        const int k4 = idx / M, m = idx % M;
        float v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int k = 4 * k4 + j;
            v[j] = (m < d_out && k < d_in) ? W[(size_t)m * d_in + k] : 0.f;
        }
        dst[idx] = make_float4(v[0], v[1], v[2], v[3]);
    }
}

cudaError_t launch_float_layer(const FloatLayerArgs &a, cudaStream_t st)
{
    if (a.n <= 0) return cudaSuccess;
    const int64_t blocks = (a.n + FTB - 1) / FTB;
    float_layer_kernel<<<(unsigned)blocks, FL_THREADS, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_prep_float_weights(const float *W, int d_out, int d_in, int K, int M, float *dst, cudaStream_t st)
{
    const int total = (K / 4) * M;
    prep_float_weights_kernel<<<(total + 255) / 256, 256, 0, st>>>(W, d_out, d_in, K, M, reinterpret_cast<float4 *>(dst));
    return cudaGetLastError();
}

} // namespace dhq
