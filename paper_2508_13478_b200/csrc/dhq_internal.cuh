// Host-side handle and the argument blocks passed to kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/dhq.h"
#include "dhq_math.cuh"

namespace dhq {

constexpr int kMaxLayers = 16;
constexpr int kDebugChunk = 65536; // tokens per pass of the layer-by-layer path

// Device arrays of one prepared layer.
struct LayerDev {
    int K = 0, M = 0;          // padded sizes as the definition pads them (K = 4 | w, M = w | 4)
    int Mt = 0;                // rows of the tensor-core weight tile (M rounded up to 16)
    int slab_k = 0;            // k per contiguous slab of the tensor-core image
    int d_in = 0, d_out = 0;
    int epi_mode = EPI_LINEAR;
    float phase_bound = 0.f;   // bound of |omega0 (s_w s_x acc + b)| over unsaturated inputs in [-1, 1] (prep_bound_kernel)
    float *row_l1 = nullptr;   // [M] sum_k |W_mk| + |b_m| of the unquantized row
    float *w_rot = nullptr;    // [M][K] fp32 rotated weights (kept for inspection)
    float *row_absmax = nullptr; // [M]
    int8_t *qw = nullptr;      // [M][K] codes, row-major
    uint32_t *qw_k4m = nullptr; // [K/4][M] four consecutive-k codes per word (layer-by-layer path)
    uint8_t *qw_umma = nullptr; // [Mt][K] codes in the tensor-core shared-memory image
    float *s_w = nullptr;      // [M]
    float *inv_w = nullptr;    // [M]
    float *bias = nullptr;     // [M] zero padded
    float *cA = nullptr, *cA_lo = nullptr, *cB = nullptr; // [M] epilogue constants
    uint32_t *fxP = nullptr, *fxQ = nullptr, *fxB = nullptr; // [M] fixed-point phase constants (EPI_SINE_FIXED)
    float *act = nullptr;      // [4]: frozen absmax (max taken on the bit pattern), s_x, inv, unused
    int has_uv = 0;            // two-sided transform, layer 1: l1U, l1V below
    int32_t *l1U = nullptr, *l1V = nullptr; // [M] H_M applied to u_m = q[m][0]+q[m][2] and v_m = q[m][1]+q[m][3]
    int has_f32 = 0;           // W32A32 handles keep the unquantized weights too
    float *w_f32 = nullptr;    // [K/4][M] float4: fp32 weights, zero padded (has_f32 only)
};

} // namespace dhq

struct dhq_handle_s {
    dhq_config_t cfg;
    int dims[dhq::kMaxLayers + 1];
    int L = 0, w = 0, d_L = 0;
    int device = 0;
    bool calibrated = false;
    int calib_layers_done = 0;      // layers whose per-tensor activation scale is frozen (sharded calibration)
    dhq::LayerDev layer[dhq::kMaxLayers];
    int *d_status = nullptr;        // device status word
    float *scratch[2] = {nullptr, nullptr}; // ping-pong activations of the layer-by-layer path
    int64_t scratch_tokens = 0;
    float *stage_in = nullptr, *stage_out = nullptr; // dhq_forward_host staging
    int64_t stage_tokens = 0;
    // dhq_forward_host pipeline: copy streams and events, created on first use
    static constexpr int kHostChunks = 8;
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_done = nullptr, ev_in[kHostChunks] = {}, ev_k[kHostChunks] = {};
    bool pipe_ready = false;
    int64_t launches = 0;
    void *fused = nullptr;          // state of the fused path (device parameter block)
    unsigned long long wait_limit_ns = 2000000000ull; // bound of every wait inside the fused kernel (dhq_set_wait_limit)
    bool stall_next_forward = false; // test hook: see dhq_debug_stall_next_forward
    double gabor_s0 = 0.0;          // > 0: wavelet activation (layer-by-layer path)
    int float_mode = 0;             // 0: fully quantized (DHQ); 1: W8A32 (activations fp32); 2: W32A32 (plain fp32 network)
};

namespace dhq {

// A handle's buffers live on the device that was current in dhq_prepare; a launch on another
// device with them would fault instead of returning a status, so every entry point asks first.
inline bool on_own_device(const dhq_handle_s *h)
{
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == h->device;
}

// Arguments of one pass of the layer-by-layer kernel.
struct LayerArgs {
    const float *X;        // [n][K] layer input, or NULL for layer 1 (built from coords)
    const float *coords;   // [n][2], layer 1 only
    int64_t n;
    int K, M, d_L;
    int a_bits;
    int per_token;
    int epi_mode;
    int rotate;            // 0: DHQ_ROT_NONE, the layer input is quantized as it is; 2: DHQ_ROT_BOTH (see s_w below)
    int calib_only;        // 1: only take max |rotated input| into act[0] (bit pattern max)
    const uint32_t *qw_k4m;
    const float *cA, *cA_lo, *cB;
    const uint32_t *fxP, *fxQ, *fxB;
    float *act;            // frozen absmax / s_x / inv (per-tensor mode)
    // DHQ_ROT_BOTH: raw weight scales and biases [M], omega0 and whether the layer has a sine; the
    // output is z = H_M (s_w s_x acc) + b, computed in fp64
    const float *s_w, *bias;
    double omega0;
    int sine;
    double gabor_s0;       // > 0: hidden layers apply sin(omega0 z) exp(-(s0 z)^2) instead of the sine
    float *Y;              // [n][M] or NULL
    float *out;            // [n][d_L] or NULL (last layer)
    float *dX; int8_t *dcodes; float *ds_x; int32_t *dacc; // dumps, may be NULL
};

cudaError_t launch_layer(const LayerArgs &a, cudaStream_t st);

// Arguments of one pass of the floating-point comparison datapaths (W8A32, W32A32).
struct FloatLayerArgs {
    const float *X;        // [n][K] layer input, or NULL for layer 1 (built from coords)
    const float *coords;   // [n][2], layer 1 only
    int64_t n;
    int K, M, d_L;
    int rotate;            // W8A32 with the Hadamard fold: rotate the layer input
    int w8;                // 1: quantized weights (qw_k4m, s_w); 0: fp32 weights (w_f32)
    const uint32_t *qw_k4m;
    const float4 *w_f32;
    const float *s_w, *bias;
    float omega0;
    int sine;
    float *Y;              // [n][M] or NULL
    float *out;            // [n][d_L] or NULL (last layer)
    float *dX;             // dump of the layer input, or NULL
};
cudaError_t launch_float_layer(const FloatLayerArgs &a, cudaStream_t st);
cudaError_t launch_prep_float_weights(const float *W, int d_out, int d_in, int K, int M, float *dst, cudaStream_t st);

struct PrepArgs {
    const float *W, *b;
    int d_out, d_in, K, M, Mt;
    int bits, per_channel;
    int a_bits;            // activation bit-width (enters the phase bound)
    int rotate;            // 0: DHQ_ROT_NONE, weights are quantized as they are; 2: DHQ_ROT_BOTH, columns rotated too
    int permute_rows;      // 1: rows of the tensor-core image in fused_column order (layers 2 .. L-1)
    int sine;              // hidden or first layer
    int first;             // layer 1: no phase bound from the weights (coordinates are unbounded)
    double omega0;
    LayerDev dev;
    float *phase_bound;    // device scalar
    unsigned long long *code_l1; // device scalar: sum over the layer of |q_w[m][k]| (bounds the rotated accumulators)
};
cudaError_t launch_prepare(const PrepArgs &a, cudaStream_t st, int64_t *launches);
// Epilogue constants from s_w and (per-tensor) the frozen activation scale.
cudaError_t launch_finalize(const LayerDev &dev, int a_bits, int per_token, int sine, double omega0,
                            cudaStream_t st, int64_t *launches);

// Byte offset of code (n, k) in the tensor-core shared-memory image of a weight matrix with `rows`
// rows and K codes per row.  The image is a sequence of contiguous slabs of `slab_k` consecutive
// k (all rows); inside a slab the 16-byte k-groups are the outer index and rows the inner one,
// i.e. 8-row x 16-byte core matrices stacked along rows (128 bytes apart) and along k
// (rows * 16 bytes apart) - the K-major, unswizzled operand layout of tcgen05.mma.
__host__ __device__ inline size_t umma_offset(int n, int k, int rows, int slab_k)
{
    // A 512 x 512 layer is cut once more, along its rows: eight pieces of 256 rows x 128 k (32 KB),
    // the four k-pieces of rows 0..255 first, so that the first half of the output columns can be
    // finished (and worked on) while the second half's weights still stream in.
    if (rows == 512 && slab_k == 128)
        return (size_t)((n >> 8) * 4 + k / 128) * 32768 + (size_t)((k % 128) >> 4) * 4096 + (size_t)(n & 255) * 16 + (k & 15);
    return (size_t)(k / slab_k) * rows * slab_k + (size_t)((k % slab_k) >> 4) * rows * 16 + (size_t)n * 16 + (k & 15);
}
// Codes per row in one slab: a 512 x 512 layer is streamed in slabs of 128 k (each cut in two
// 32 KB pieces of 256 rows, see umma_offset); narrower layers are one slab.
__host__ __device__ inline int fused_slab_k(int K, int rows) { return (K == 512 && rows == 512) ? 128 : (K < 16 ? 16 : K); }
// Columns of a hidden layer's output are processed by the fused kernel in register chunks of
// fused_chunk(W) columns, and inside a chunk the features i and i + chunk/2 sit in adjacent
// tensor-memory columns (2i, 2i+1) so that they form the two halves of a packed fp32x2 register.
// fused_column(m, W) is the tensor-memory column (= row of the weight image) of output feature m.
__host__ __device__ inline int fused_chunk(int W) { return W == 64 ? 32 : 64; }
__host__ __device__ inline int fused_column(int m, int W)
{
    const int ch = fused_chunk(W), c = m / ch, f = m % ch;
    return c * ch + (f < ch / 2 ? 2 * f : 2 * (f - ch / 2) + 1);
}
__host__ __device__ inline int fused_feature(int col, int W)
{
    const int ch = fused_chunk(W), c = col / ch, j = col % ch;
    return c * ch + (j >> 1) + (j & 1) * (ch / 2);
}
// Fused tensor-core forward.
dhq_status_t fused_create(dhq_handle_s *h);
void fused_destroy(dhq_handle_s *h);
// on_host: coords / out are device aliases of mapped host memory (the variants that fetch the next
// tile's coordinates early are for device memory)
dhq_status_t fused_forward(dhq_handle_s *h, const float *coords, int64_t n, float *out, bool on_host, cudaStream_t st);
// Per-layer dump targets of the observing instantiation of the fused kernel: device pointers
// laid out as dhq_debug_bufs_t describes, entry l-1 for layer l, NULL entries skipped.  X is only
// used for layer 1; the input of a later layer is the output of the one before it.
// One calibration pass of layer l (1-based) by the fused kernel; needs a fused handle with per-tensor
// activation scales and not the two-sided transform.
dhq_status_t fused_calibrate_layer(dhq_handle_s *h, int l, const float *coords, int64_t n, cudaStream_t st);
struct DumpPtrs {
    float *X[kMaxLayers];
    int8_t *codes[kMaxLayers];
    float *s_x[kMaxLayers];
    int32_t *acc[kMaxLayers];
    float *Y[kMaxLayers];
};
dhq_status_t fused_forward_dump(dhq_handle_s *h, const float *coords, int64_t n, float *out, const DumpPtrs &d, cudaStream_t st);
// Coordinates one launch of the fused kernel works on at a time over the whole GPU (one tile per
// slot of every SM): launches cut at multiples of this leave no SM idle.
int64_t fused_round_tokens(const dhq_handle_s *h);
// The fused kernel's per-element loops of a width-256 hidden layer in isolation (micro-benchmark):
// which = 1 pass 1, 2 pass 2, 3 both; one block of 16 warps on each of `sms` SMs.  Each iteration
// covers 256 tokens x 256 activation elements per SM.
cudaError_t launch_pass_rate(int which, int sms, int iters, cudaStream_t st);

} // namespace dhq
