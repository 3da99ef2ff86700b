// C ABI of the library (see include/dhq.h): argument checks, the handle, and the sequencing of
// kernels on the caller's stream.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include "dhq_internal.cuh"

using namespace dhq;

#define CK(call)                                         \
    do {                                                 \
        cudaError_t e_ = (call);                         \
        if (e_ != cudaSuccess) return DHQ_ERR_CUDA;      \
    } while (0)

namespace {

template <typename T> bool dev_alloc(T **p, size_t count)
{
    return cudaMalloc((void **)p, count * sizeof(T) < 16 ? 16 : count * sizeof(T)) == cudaSuccess;
}

// Every device array of a prepared layer with its size in bytes, in a fixed order (allocation,
// release, export and import all walk this table).  Needs d.K, d.M, d.Mt.
struct ArrayRef { void **ptr; size_t bytes; };
constexpr int kLayerArrays = 19;
void layer_arrays(LayerDev &d, ArrayRef (&t)[kLayerArrays])
{
    const size_t MK = (size_t)d.M * d.K, M = (size_t)d.M;
    int i = 0;
    t[i++] = {(void **)&d.w_rot, MK * 4};
    t[i++] = {(void **)&d.row_absmax, M * 4};
    t[i++] = {(void **)&d.row_l1, M * 4};
    t[i++] = {(void **)&d.qw, MK};
    t[i++] = {(void **)&d.qw_k4m, MK};
    t[i++] = {(void **)&d.qw_umma, (size_t)d.Mt * (d.K < 16 ? 16 : d.K)};
    t[i++] = {(void **)&d.s_w, M * 4};
    t[i++] = {(void **)&d.inv_w, M * 4};
    t[i++] = {(void **)&d.bias, M * 4};
    t[i++] = {(void **)&d.cA, M * 4};
    t[i++] = {(void **)&d.cA_lo, M * 4};
    t[i++] = {(void **)&d.cB, M * 4};
    t[i++] = {(void **)&d.fxP, M * 4};
    t[i++] = {(void **)&d.fxQ, M * 4};
    t[i++] = {(void **)&d.fxB, M * 4};
    t[i++] = {(void **)&d.act, 16};
    t[i++] = {(void **)&d.w_f32, d.has_f32 ? MK * 4 : 0};
    t[i++] = {(void **)&d.l1U, d.has_uv ? M * 4 : 0};
    t[i++] = {(void **)&d.l1V, d.has_uv ? M * 4 : 0};
}

bool alloc_layer(LayerDev &d)
{
    ArrayRef t[kLayerArrays];
    layer_arrays(d, t);
    for (const ArrayRef &a : t)
        if (cudaMalloc(a.ptr, a.bytes < 16 ? 16 : a.bytes) != cudaSuccess) return false;
    return true;
}

void free_layer(LayerDev &d)
{
    ArrayRef t[kLayerArrays];
    layer_arrays(d, t);
    for (const ArrayRef &a : t) cudaFree(*a.ptr);
    d = LayerDev();
}

// Padded sizes of layer l (1-based) of a network of hidden width w.
void set_layer_dims(LayerDev &d, int l, int L, int w, const int *dims)
{
    d.K = (l == 1) ? 4 : w;
    d.M = (l == L) ? 4 : w;
    d.Mt = d.M < 16 ? 16 : d.M;
    d.slab_k = fused_slab_k(d.K, d.Mt);
    d.d_in = dims[l - 1];
    d.d_out = dims[l];
}

dhq_status_t check_config(const dhq_config_t *cfg)
{
    const int L = cfg->n_layers;
    if (L < 2 || L > kMaxLayers) return DHQ_ERR_INVALID_ARG;
    const int w = cfg->dims[1], d_L = cfg->dims[L];
    if (cfg->dims[0] != 2 || w <= 0 || (w & (w - 1)) != 0 || w < 64 || w > 512 || d_L < 1 || d_L > 4) return DHQ_ERR_UNSUPPORTED;
    for (int l = 1; l < L; ++l)
        if (cfg->dims[l] != w) return DHQ_ERR_UNSUPPORTED;
    const bool wq = cfg->w_bits >= 2 && cfg->w_bits <= 8, aq = cfg->a_bits >= 2 && cfg->a_bits <= 8;
    const bool wf = cfg->w_bits == DHQ_BITS_FLOAT, af = cfg->a_bits == DHQ_BITS_FLOAT;
    if (!((wq && aq) || (wq && af) || (wf && af))) return DHQ_ERR_UNSUPPORTED; // W8A8 family, W8A32 family, W32A32
    if (cfg->rotation != DHQ_ROT_INPUT && cfg->rotation != DHQ_ROT_NONE && cfg->rotation != DHQ_ROT_BOTH) return DHQ_ERR_UNSUPPORTED;
    if (af && cfg->rotation == DHQ_ROT_BOTH) return DHQ_ERR_UNSUPPORTED;
    if (cfg->activation != DHQ_ACT_SINE && cfg->activation != DHQ_ACT_GABOR) return DHQ_ERR_UNSUPPORTED;
    if (cfg->activation == DHQ_ACT_GABOR) {
        if (af) return DHQ_ERR_UNSUPPORTED;
        if (!(cfg->act_s0 > 0.0f) || std::isinf(cfg->act_s0) || cfg->omega0 == 0.0f) return DHQ_ERR_INVALID_ARG;
    }
    if ((cfg->w_gran != DHQ_GRAN_TENSOR && cfg->w_gran != DHQ_GRAN_CHANNEL_OR_TOKEN) ||
        (cfg->a_gran != DHQ_GRAN_TENSOR && cfg->a_gran != DHQ_GRAN_CHANNEL_OR_TOKEN))
        return DHQ_ERR_INVALID_ARG;
    if (!(cfg->omega0 == cfg->omega0) || std::isinf(cfg->omega0)) return DHQ_ERR_INVALID_ARG;
    return DHQ_OK;
}

// Which datapath a configuration asks for: 0 fully quantized, 1 W8A32, 2 W32A32.
int float_mode_of(const dhq_config_t &cfg)
{
    if (cfg.a_bits != DHQ_BITS_FLOAT) return 0;
    return cfg.w_bits == DHQ_BITS_FLOAT ? 2 : 1;
}

// Serialized handle (dhq_export / dhq_import): this header, then every array of every layer in
// the order of layer_arrays.
struct BlobHeader {
    char magic[8];            // "DHQB200\0"
    uint32_t version, header_bytes;
    int32_t n_layers, dims[kMaxLayers + 1];
    int32_t w_bits, a_bits, w_gran, a_gran, rotation, activation;
    float omega0, act_s0;
    int32_t calibrated, calib_layers_done, has_fused;
    int32_t epi_mode[kMaxLayers];
    float phase_bound[kMaxLayers];
    uint64_t payload_bytes, payload_fnv1a;
};
constexpr uint32_t kBlobVersion = 4;
const char kBlobMagic[8] = {'D', 'H', 'Q', 'B', '2', '0', '0', 0};

uint64_t fnv1a(const uint8_t *p, size_t n)
{
    uint64_t hsh = 1469598103934665603ull;
    for (size_t i = 0; i < n; ++i) hsh = (hsh ^ p[i]) * 1099511628211ull;
    return hsh;
}


dhq_status_t ensure_scratch(dhq_handle_s *h, int64_t tokens)
{
    if (tokens <= h->scratch_tokens) return DHQ_OK;
    CK(cudaDeviceSynchronize());
    cudaFree(h->scratch[0]); cudaFree(h->scratch[1]);
    h->scratch[0] = h->scratch[1] = nullptr;
    h->scratch_tokens = 0;
    for (int i = 0; i < 2; ++i)
        if (!dev_alloc(&h->scratch[i], (size_t)tokens * h->w)) return DHQ_ERR_ALLOC;
    h->scratch_tokens = tokens;
    return DHQ_OK;
}

// Arguments of layer l (1-based) over tokens [t0, t0+cnt) with the given input/output buffers.
LayerArgs layer_args(dhq_handle_s *h, int l, const float *coords, const float *X, int64_t cnt)
{
    const LayerDev &d = h->layer[l - 1];
    LayerArgs a;
    memset(&a, 0, sizeof(a));
    a.X = X; a.coords = coords; a.n = cnt;
    a.K = d.K; a.M = d.M; a.d_L = h->d_L;
    a.a_bits = h->cfg.a_bits;
    a.per_token = h->cfg.a_gran == DHQ_GRAN_CHANNEL_OR_TOKEN;
    a.epi_mode = d.epi_mode;
    a.rotate = h->cfg.rotation == DHQ_ROT_INPUT ? 1 : h->cfg.rotation == DHQ_ROT_BOTH ? 2 : 0;
    a.s_w = d.s_w; a.bias = d.bias; a.omega0 = (double)h->cfg.omega0; a.sine = l < h->L;
    a.gabor_s0 = h->gabor_s0;
    a.qw_k4m = d.qw_k4m; a.cA = d.cA; a.cA_lo = d.cA_lo; a.cB = d.cB; a.act = d.act;
    a.fxP = d.fxP; a.fxQ = d.fxQ; a.fxB = d.fxB;
    return a;
}

// One calibration pass: the maximum of |rotated input of layer l| over the given coordinates, with
// layers < l run as they are frozen, is left in the layer's act[0] (not yet turned into scales).
dhq_status_t calibrate_layer_pass(dhq_handle_s *h, int l, const float *coords, int64_t n, cudaStream_t st)
{
    if (h->fused && ((uintptr_t)coords & 7) == 0) {
        // the fused kernel run up to layer l's rotated input: one launch instead of l layer passes per
        // 64 Ki coordinates; same arithmetic, so the same maximum bit for bit
        CK(cudaMemsetAsync(h->layer[l - 1].act, 0, 4 * sizeof(float), st));
        return fused_calibrate_layer(h, l, coords, n, st);
    }
    const int64_t chunk = n < kDebugChunk ? n : kDebugChunk;
    dhq_status_t s = ensure_scratch(h, chunk);
    if (s != DHQ_OK) return s;
    LayerDev &d = h->layer[l - 1];
    CK(cudaMemsetAsync(d.act, 0, 4 * sizeof(float), st));
    for (int64_t t0 = 0; t0 < n; t0 += chunk) {
        int64_t cnt = n - t0 < chunk ? n - t0 : chunk;
        const float *X = nullptr;
        for (int j = 1; j <= l; ++j) {
            LayerArgs a = layer_args(h, j, coords + t0 * 2, X, cnt);
            if (j == l) a.calib_only = 1;
            else a.Y = h->scratch[(j - 1) & 1];
            CK(launch_layer(a, st));
            h->launches++;
            X = a.Y;
        }
    }
    return DHQ_OK;
}

dhq_status_t calibrate_impl(dhq_handle_s *h, const float *coords, int64_t n, cudaStream_t st)
{
    for (int l = 1; l <= h->L; ++l) {
        dhq_status_t s = calibrate_layer_pass(h, l, coords, n, st);
        if (s != DHQ_OK) return s;
        CK(launch_finalize(h->layer[l - 1], h->cfg.a_bits, 0, l < h->L, (double)h->cfg.omega0, st, &h->launches));
    }
    h->calibrated = true;
    h->calib_layers_done = h->L;
    return DHQ_OK;
}

// Layers 1..L one kernel pass each over tokens in chunks, activations in the handle's scratch.
dhq_status_t layerwise_forward(dhq_handle_s *h, const float *coords, int64_t n, float *out, cudaStream_t st)
{
    const int64_t chunk = n < kDebugChunk ? n : kDebugChunk;
    dhq_status_t s = ensure_scratch(h, chunk);
    if (s != DHQ_OK) return s;
    for (int64_t t0 = 0; t0 < n; t0 += chunk) {
        int64_t cnt = n - t0 < chunk ? n - t0 : chunk;
        const float *X = nullptr;
        for (int l = 1; l <= h->L; ++l) {
            LayerArgs a = layer_args(h, l, coords + t0 * 2, X, cnt);
            a.Y = h->scratch[(l - 1) & 1];
            if (l == h->L) a.out = out + t0 * h->d_L;
            CK(launch_layer(a, st));
            h->launches++;
            X = a.Y;
        }
    }
    return DHQ_OK;
}

// W8A32 / W32A32: one pass of the floating-point layer kernel per layer, in chunks; X dumps optional.
dhq_status_t float_forward(dhq_handle_s *h, const float *coords, int64_t n, float *out, const dhq_debug_bufs_t *bufs, cudaStream_t st)
{
    const int64_t chunk = n < kDebugChunk ? n : kDebugChunk;
    dhq_status_t s = ensure_scratch(h, chunk);
    if (s != DHQ_OK) return s;
    for (int64_t t0 = 0; t0 < n; t0 += chunk) {
        const int64_t cnt = n - t0 < chunk ? n - t0 : chunk;
        const float *X = nullptr;
        for (int l = 1; l <= h->L; ++l) {
            const LayerDev &d = h->layer[l - 1];
            FloatLayerArgs a;
            memset(&a, 0, sizeof(a));
            a.X = X; a.coords = coords + t0 * 2; a.n = cnt;
            a.K = d.K; a.M = d.M; a.d_L = h->d_L;
            a.w8 = h->float_mode == 1;
            a.rotate = a.w8 && h->cfg.rotation == DHQ_ROT_INPUT;
            a.qw_k4m = d.qw_k4m; a.w_f32 = reinterpret_cast<const float4 *>(d.w_f32);
            a.s_w = d.s_w; a.bias = d.bias;
            a.omega0 = h->cfg.omega0; a.sine = l < h->L;
            a.Y = h->scratch[(l - 1) & 1];
            if (l == h->L) a.out = out ? out + t0 * h->d_L : nullptr;
            if (bufs) {
                if (bufs->X && bufs->X[l - 1]) a.dX = bufs->X[l - 1] + t0 * d.K;
                if (bufs->Y && bufs->Y[l - 1]) a.Y = bufs->Y[l - 1] + t0 * d.M;
            }
            CK(launch_float_layer(a, st));
            h->launches++;
            X = a.Y;
        }
    }
    return DHQ_OK;
}

// The forward pass of a calibrated handle: the fused kernel, or, for the two-sided transform, the
// layer-by-layer kernels.
dhq_status_t run_forward(dhq_handle_s *h, const float *coords, int64_t n, float *out, bool on_host, cudaStream_t st)
{
    if (h->float_mode) return float_forward(h, coords, n, out, nullptr, st);
    if (!h->fused) return layerwise_forward(h, coords, n, out, st); // wavelet activation; two-sided transform with per-channel weight scales
    return fused_forward(h, coords, n, out, on_host, st);
}

} // namespace

extern "C" {

const char *dhq_status_string(dhq_status_t s)
{
    switch (s) {
    case DHQ_OK: return "ok";
    case DHQ_ERR_INVALID_ARG: return "invalid argument";
    case DHQ_ERR_UNSUPPORTED: return "unsupported shape or option";
    case DHQ_ERR_ALLOC: return "allocation failed";
    case DHQ_ERR_CUDA: return "CUDA runtime error";
    case DHQ_ERR_NOT_CALIBRATED: return "per-tensor activation scales are not calibrated";
    case DHQ_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case DHQ_ERR_TOO_LARGE: return "more tokens than the fixed-size scratch area holds";
    }
    return "unknown status";
}

void dhq_destroy(dhq_handle_t h)
{
    if (!h) return;
    cudaDeviceSynchronize();
    fused_destroy(h);
    for (int l = 0; l < kMaxLayers; ++l) free_layer(h->layer[l]);
    cudaFree(h->d_status);
    cudaFree(h->scratch[0]); cudaFree(h->scratch[1]);
    cudaFree(h->stage_in); cudaFree(h->stage_out);
    if (h->copy_in) cudaStreamDestroy(h->copy_in);
    if (h->copy_out) cudaStreamDestroy(h->copy_out);
    if (h->ev_start) cudaEventDestroy(h->ev_start);
    if (h->ev_done) cudaEventDestroy(h->ev_done);
    for (int i = 0; i < dhq_handle_s::kHostChunks; ++i) {
        if (h->ev_in[i]) cudaEventDestroy(h->ev_in[i]);
        if (h->ev_k[i]) cudaEventDestroy(h->ev_k[i]);
    }
    delete h;
}

static dhq_status_t prepare_impl(const dhq_config_t *cfg, const float *const *W, const float *const *b,
                                 void *stream, dhq_handle_t *out)
{
    if (!cfg || !W || !b || !out || !cfg->dims) return DHQ_ERR_INVALID_ARG;
    *out = nullptr;
    const int L = cfg->n_layers;
    if (L < 2 || L > kMaxLayers) return DHQ_ERR_INVALID_ARG;
    for (int l = 0; l < L; ++l)
        if (!W[l] || !b[l]) return DHQ_ERR_INVALID_ARG;
    {
        dhq_status_t cs = check_config(cfg);
        if (cs != DHQ_OK) return cs;
    }
    const int w = cfg->dims[1], d_L = cfg->dims[L];

    dhq_handle_s *h = new (std::nothrow) dhq_handle_s();
    if (!h) return DHQ_ERR_ALLOC;
    h->cfg = *cfg;
    for (int i = 0; i <= L; ++i) h->dims[i] = cfg->dims[i];
    h->cfg.dims = h->dims;
    h->L = L; h->w = w; h->d_L = d_L;
    cudaStream_t st = (cudaStream_t)stream;
    dhq_status_t rc = DHQ_OK;
    float *d_bounds = nullptr;
    unsigned long long *d_sums = nullptr;
    const bool both = cfg->rotation == DHQ_ROT_BOTH;
    h->float_mode = float_mode_of(*cfg);
    h->gabor_s0 = cfg->activation == DHQ_ACT_GABOR ? (double)cfg->act_s0 : 0.0;
    const bool gabor = h->gabor_s0 > 0.0;
    // the floating-point datapaths have no activation quantizer: nothing to calibrate
    const bool per_token = cfg->a_gran == DHQ_GRAN_CHANNEL_OR_TOKEN || h->float_mode != 0;
    do {
        if (cudaGetDevice(&h->device) != cudaSuccess) { rc = DHQ_ERR_CUDA; break; }
        if (!dev_alloc(&h->d_status, 16) || !dev_alloc(&d_bounds, kMaxLayers) || !dev_alloc(&d_sums, kMaxLayers)) { rc = DHQ_ERR_ALLOC; break; }
        if (cudaMemsetAsync(h->d_status, 0, 64, st) != cudaSuccess ||
            cudaMemsetAsync(d_bounds, 0, kMaxLayers * sizeof(float), st) != cudaSuccess ||
            cudaMemsetAsync(d_sums, 0, kMaxLayers * sizeof(unsigned long long), st) != cudaSuccess) { rc = DHQ_ERR_CUDA; break; }
        for (int l = 1; l <= L && rc == DHQ_OK; ++l) {
            LayerDev &d = h->layer[l - 1];
            set_layer_dims(d, l, L, w, cfg->dims);
            // coordinates are not bounded by the weights; the wavelet's envelope needs the unwrapped phase
            if (l == 1) d.epi_mode = (per_token || gabor) ? EPI_SINE_WIDE : EPI_SINE_FIXED;
            d.has_uv = both && l == 1;
            d.has_f32 = h->float_mode == 2;
            if (!alloc_layer(d)) { rc = DHQ_ERR_ALLOC; break; }
            if (d.has_f32 && launch_prep_float_weights(W[l - 1], d.d_out, d.d_in, d.K, d.M, d.w_f32, st) != cudaSuccess) {
                rc = DHQ_ERR_CUDA; break;
            }
            if (cudaMemsetAsync(d.act, 0, 16, st) != cudaSuccess) { rc = DHQ_ERR_CUDA; break; }
            PrepArgs a;
            memset(&a, 0, sizeof(a));
            a.W = W[l - 1]; a.b = b[l - 1];
            a.d_out = d.d_out; a.d_in = d.d_in; a.K = d.K; a.M = d.M; a.Mt = d.Mt;
            // (a W32A32 handle still gets 8-bit codes of the unrotated weights; its forward does not read them)
            a.bits = h->float_mode == 2 ? 8 : cfg->w_bits;
            a.a_bits = h->float_mode ? 8 : cfg->a_bits;
            a.per_channel = cfg->w_gran == DHQ_GRAN_CHANNEL_OR_TOKEN;
            a.sine = l < L; a.first = l == 1;
            a.permute_rows = (l > 1 && l < L) ? 1 : 0;
            a.rotate = h->float_mode == 2 ? 0 : cfg->rotation == DHQ_ROT_INPUT ? 1 : both ? 2 : 0;
            a.omega0 = (double)cfg->omega0;
            a.dev = d;
            a.phase_bound = d_bounds + (l - 1);
            a.code_l1 = d_sums + (l - 1);
            if (launch_prepare(a, st, &h->launches) != cudaSuccess) { rc = DHQ_ERR_CUDA; break; }
            if (per_token &&
                launch_finalize(d, h->float_mode ? 8 : cfg->a_bits, 1, l < L, (double)cfg->omega0, st, &h->launches) != cudaSuccess) {
                rc = DHQ_ERR_CUDA; break;
            }
        }
        if (rc != DHQ_OK) break;
        float bounds[kMaxLayers];
        unsigned long long sums[kMaxLayers];
        if (cudaMemcpyAsync(bounds, d_bounds, sizeof(bounds), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaMemcpyAsync(sums, d_sums, sizeof(sums), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess) { rc = DHQ_ERR_CUDA; break; }
        // Two-sided transform in the fused kernel: the output-side rotation runs on the int32 accumulators,
        // which needs one weight scale per tensor and |H_M acc| <= sum_m |acc_m| <= qmax_a * sum |q_w| < 2^31.
        bool both_fused = both && cfg->w_gran == DHQ_GRAN_TENSOR && !h->float_mode;
        for (int l = 1; l <= L && both_fused; ++l)
            if (sums[l - 1] * (unsigned long long)((1 << (cfg->a_bits - 1)) - 1) >= (1ull << 31)) both_fused = false;
        const bool a_per_token = cfg->a_gran == DHQ_GRAN_CHANNEL_OR_TOKEN;
        for (int l = 1; l <= L; ++l) {
            LayerDev &d = h->layer[l - 1];
            d.phase_bound = bounds[l - 1];
            if (l == L) d.epi_mode = EPI_LINEAR;
            else if (l == 1) {}
            // (two-sided: the quantization error of all M rows meets in every output; no tight phase bound)
            else if (bounds[l - 1] <= (a_per_token ? kFastPhaseLimitPerToken : kFastPhaseLimit) && !gabor && !both) d.epi_mode = EPI_SINE_FAST;
            // no bound below the limit: the values that are below it still take the short route (the kernels
            // with a per-token scale and the fused two-sided ones carry that variant)
            else d.epi_mode = (!gabor && !h->float_mode && ((a_per_token && !both) || both_fused)) ? EPI_SINE_MIXED : EPI_SINE_WIDE;
        }
        h->calibrated = per_token;
        // layer by layer: the fp32 datapaths, the two-sided transform with per-channel weight scales, and the
        // wavelet combined with the two-sided transform
        if ((!both || both_fused) && !h->float_mode) rc = fused_create(h);
    } while (0);
    cudaFree(d_bounds);
    cudaFree(d_sums);
    if (rc != DHQ_OK) {
        dhq_destroy(h);
        return rc;
    }
    *out = h;
    return DHQ_OK;
}

static dhq_status_t calibrate_entry(dhq_handle_t h, const float *coords, int64_t n, void *stream)
{
    if (!h || !coords || n < 1) return DHQ_ERR_INVALID_ARG;
    if (!on_own_device(h)) return DHQ_ERR_INVALID_ARG;
    if (h->cfg.a_gran == DHQ_GRAN_CHANNEL_OR_TOKEN || h->float_mode) return DHQ_OK;
    return calibrate_impl(h, coords, n, (cudaStream_t)stream);
}

dhq_status_t dhq_calibrate_layer(dhq_handle_t h, int layer, const float *coords, int64_t n, void *stream)
{
    if (!h || layer < 1 || layer > h->L || n < 0 || (n > 0 && !coords)) return DHQ_ERR_INVALID_ARG;
    if (!on_own_device(h)) return DHQ_ERR_INVALID_ARG;
    if (h->cfg.a_gran == DHQ_GRAN_CHANNEL_OR_TOKEN || h->float_mode) return DHQ_OK;
    if (layer > h->calib_layers_done + 1) return DHQ_ERR_NOT_CALIBRATED; // layers before it are not frozen yet
    h->calibrated = false;
    h->calib_layers_done = layer - 1;
    if (n == 0) { // a rank without coordinates contributes the neutral element
        CK(cudaMemsetAsync(h->layer[layer - 1].act, 0, 4 * sizeof(float), (cudaStream_t)stream));
        return DHQ_OK;
    }
    return calibrate_layer_pass(h, layer, coords, n, (cudaStream_t)stream);
}

dhq_status_t dhq_get_act_absmax(dhq_handle_t h, int layer, float *absmax, void *stream)
{
    if (!h || layer < 1 || layer > h->L || !absmax) return DHQ_ERR_INVALID_ARG;
    if (!on_own_device(h)) return DHQ_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    CK(cudaMemcpyAsync(absmax, h->layer[layer - 1].act, sizeof(float), cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
    return DHQ_OK;
}

dhq_status_t dhq_set_act_absmax(dhq_handle_t h, int layer, float absmax, void *stream)
{
    if (!h || layer < 1 || layer > h->L || !(absmax >= 0.0f) || std::isinf(absmax)) return DHQ_ERR_INVALID_ARG;
    if (!on_own_device(h)) return DHQ_ERR_INVALID_ARG;
    if (h->cfg.a_gran == DHQ_GRAN_CHANNEL_OR_TOKEN || h->float_mode) return DHQ_OK;
    if (layer > h->calib_layers_done + 1) return DHQ_ERR_NOT_CALIBRATED;
    cudaStream_t st = (cudaStream_t)stream;
    CK(cudaMemcpyAsync(h->layer[layer - 1].act, &absmax, sizeof(float), cudaMemcpyHostToDevice, st));
    CK(cudaStreamSynchronize(st)); // `absmax` lives on this call's stack
    CK(launch_finalize(h->layer[layer - 1], h->cfg.a_bits, 0, layer < h->L, (double)h->cfg.omega0, st, &h->launches));
    h->calib_layers_done = layer;
    h->calibrated = layer == h->L;
    return DHQ_OK;
}

dhq_status_t dhq_forward_debug(dhq_handle_t h, const float *coords, int64_t n, float *out,
                               const dhq_debug_bufs_t *bufs, void *stream)
{
    if (!h || n < 0 || (n > 0 && !coords)) return DHQ_ERR_INVALID_ARG;
    if (!on_own_device(h)) return DHQ_ERR_INVALID_ARG;
    if (n == 0) return DHQ_OK;
    if (h->float_mode) return float_forward(h, coords, n, out, bufs, (cudaStream_t)stream); // X and Y dumps only
    if (!h->calibrated) return DHQ_ERR_NOT_CALIBRATED;
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t chunk = n < kDebugChunk ? n : kDebugChunk;
    dhq_status_t s = ensure_scratch(h, chunk);
    if (s != DHQ_OK) return s;
    for (int64_t t0 = 0; t0 < n; t0 += chunk) {
        int64_t cnt = n - t0 < chunk ? n - t0 : chunk;
        const float *X = nullptr;
        for (int l = 1; l <= h->L; ++l) {
            const LayerDev &d = h->layer[l - 1];
            LayerArgs a = layer_args(h, l, coords + t0 * 2, X, cnt);
            a.Y = h->scratch[(l - 1) & 1];
            if (l == h->L) a.out = out ? out + t0 * h->d_L : nullptr;
            if (bufs) {
                if (bufs->X && bufs->X[l - 1]) a.dX = bufs->X[l - 1] + t0 * d.K;
                if (bufs->codes && bufs->codes[l - 1]) a.dcodes = bufs->codes[l - 1] + t0 * d.K;
                if (bufs->s_x && bufs->s_x[l - 1]) a.ds_x = bufs->s_x[l - 1] + t0;
                if (bufs->acc && bufs->acc[l - 1]) a.dacc = bufs->acc[l - 1] + t0 * d.M;
                if (bufs->Y && bufs->Y[l - 1]) a.Y = bufs->Y[l - 1] + t0 * d.M;
            }
            CK(launch_layer(a, st));
            h->launches++;
            X = a.Y;
        }
    }
    return DHQ_OK;
}

dhq_status_t dhq_forward_fused_debug(dhq_handle_t h, const float *coords, int64_t n, float *out,
                                     const dhq_debug_bufs_t *bufs, void *stream)
{
    if (!h || n < 0 || (n > 0 && (!coords || !out))) return DHQ_ERR_INVALID_ARG;
    if (!on_own_device(h)) return DHQ_ERR_INVALID_ARG;
    if (n == 0) return DHQ_OK;
    if (((uintptr_t)coords & 7) || ((uintptr_t)out & 3)) return DHQ_ERR_INVALID_ARG;
    if (!h->fused) return DHQ_ERR_UNSUPPORTED; // this handle runs layer by layer: dhq_forward_debug
    if (!h->calibrated) return DHQ_ERR_NOT_CALIBRATED;
    cudaStream_t st = (cudaStream_t)stream;
    DumpPtrs d;
    memset(&d, 0, sizeof(d));
    if (bufs) {
        for (int l = 1; l <= h->L; ++l) {
            if (bufs->codes && bufs->codes[l - 1]) d.codes[l - 1] = bufs->codes[l - 1];
            if (bufs->s_x && bufs->s_x[l - 1]) d.s_x[l - 1] = bufs->s_x[l - 1];
            if (bufs->acc && bufs->acc[l - 1]) d.acc[l - 1] = bufs->acc[l - 1];
            if (bufs->Y && bufs->Y[l - 1]) d.Y[l - 1] = bufs->Y[l - 1];
        }
        if (bufs->X && bufs->X[0]) d.X[0] = bufs->X[0];
        // inside the fused kernel the input of layer l+1 IS the output of layer l (one value, in
        // registers): it is written once, to Y[l-1] if given, else straight to X[l]
        for (int l = 1; l < h->L; ++l)
            if (!d.Y[l - 1] && bufs->X && bufs->X[l]) d.Y[l - 1] = bufs->X[l];
        if (((uintptr_t)d.X[0] & 15)) return DHQ_ERR_INVALID_ARG;
        for (int l = 0; l < h->L; ++l)
            if (((uintptr_t)d.codes[l] & 3) || ((uintptr_t)d.s_x[l] & 3) || ((uintptr_t)d.acc[l] & 3) || ((uintptr_t)d.Y[l] & 3))
                return DHQ_ERR_INVALID_ARG;
    }
    dhq_status_t s = fused_forward_dump(h, coords, n, out, d, st);
    if (s != DHQ_OK) return s;
    if (bufs && bufs->X)
        for (int l = 1; l < h->L; ++l)
            if (bufs->X[l] && d.Y[l - 1] != bufs->X[l])
                CK(cudaMemcpyAsync(bufs->X[l], d.Y[l - 1], (size_t)n * h->w * sizeof(float), cudaMemcpyDeviceToDevice, st));
    return DHQ_OK;
}

dhq_status_t dhq_set_wait_limit(dhq_handle_t h, int64_t nanoseconds)
{
    if (!h || nanoseconds < 1000) return DHQ_ERR_INVALID_ARG;
    h->wait_limit_ns = (unsigned long long)nanoseconds;
    return DHQ_OK;
}

dhq_status_t dhq_debug_stall_next_forward(dhq_handle_t h)
{
    if (!h) return DHQ_ERR_INVALID_ARG;
    if (!h->fused) return DHQ_ERR_UNSUPPORTED;
    h->stall_next_forward = true;
    return DHQ_OK;
}

static dhq_status_t forward_entry(dhq_handle_t h, const float *coords, int64_t n, float *out, void *stream)
{
    if (!h || n < 0 || (n > 0 && (!coords || !out))) return DHQ_ERR_INVALID_ARG;
    if (!on_own_device(h)) return DHQ_ERR_INVALID_ARG;
    if (n == 0) return DHQ_OK;
    if (((uintptr_t)coords & 7) || ((uintptr_t)out & 3)) return DHQ_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (!h->calibrated) {
        dhq_status_t s = calibrate_impl(h, coords, n, st);
        if (s != DHQ_OK) return s;
    }
    return run_forward(h, coords, n, out, false, st);
}

static dhq_status_t forward_host_entry(dhq_handle_t h, const float *coords_host, int64_t n, float *out_host,
                                       void *stream)
{
    if (!h || n < 0 || (n > 0 && (!coords_host || !out_host))) return DHQ_ERR_INVALID_ARG;
    if (!on_own_device(h)) return DHQ_ERR_INVALID_ARG;
    if (n == 0) return DHQ_OK;
    cudaStream_t st = (cudaStream_t)stream;
    // Pinned (page-locked, device-mapped) host buffers need no staging: the fused kernel reads the
    // coordinates and writes the result through their device addresses, so the transfers happen
    // inside the kernel, tile by tile, beside the arithmetic.  (Calibration reads the coordinates
    // once per layer: it goes through the staged path below.)
    if (h->calibrated && h->fused && !((uintptr_t)coords_host & 7) && !((uintptr_t)out_host & 3)) {
        // one query per buffer: for page-locked memory it also gives the device alias (asked on every
        // call on purpose: an answer remembered per address could outlive the buffer it was given for)
        cudaPointerAttributes ai, ao;
        const bool mapped = cudaPointerGetAttributes(&ai, coords_host) == cudaSuccess && ai.type == cudaMemoryTypeHost &&
                            cudaPointerGetAttributes(&ao, out_host) == cudaSuccess && ao.type == cudaMemoryTypeHost &&
                            ai.devicePointer && ao.devicePointer;
        void *di = mapped ? ai.devicePointer : nullptr, *dout = mapped ? ao.devicePointer : nullptr;
        (void)cudaGetLastError(); // a failed query of pageable memory is not an error of this call
        if (mapped) return run_forward(h, static_cast<const float *>(di), n, static_cast<float *>(dout), true, st);
    }
    if (n > h->stage_tokens) {
        CK(cudaDeviceSynchronize());
        cudaFree(h->stage_in); cudaFree(h->stage_out);
        h->stage_in = h->stage_out = nullptr;
        h->stage_tokens = 0;
        if (!dev_alloc(&h->stage_in, (size_t)n * 2) || !dev_alloc(&h->stage_out, (size_t)n * h->d_L))
            return DHQ_ERR_ALLOC;
        h->stage_tokens = n;
    }
    // How many launches the call is cut into: each is a whole number of rounds of the fused kernel
    // (one tile per slot of every SM), so that cutting costs only the launch prologue.
    const int64_t round = fused_round_tokens(h);
    const int64_t rounds = (n + round - 1) / round;
    int chunks = (int)(rounds >= 16 ? 8 : rounds < 4 ? rounds : 4);
    if (!h->calibrated || !h->fused) chunks = 1; // the first forward freezes the per-tensor
                                                                 // scales on ALL of its coordinates; the layer-by-layer paths are not cut
    if (chunks <= 1) {
        CK(cudaMemcpyAsync(h->stage_in, coords_host, (size_t)n * 2 * sizeof(float), cudaMemcpyHostToDevice, st));
        dhq_status_t s = forward_entry(h, h->stage_in, n, h->stage_out, stream);
        if (s != DHQ_OK) return s;
        CK(cudaMemcpyAsync(out_host, h->stage_out, (size_t)n * h->d_L * sizeof(float), cudaMemcpyDeviceToHost, st));
        return DHQ_OK;
    }
    // Pipeline: the copy of chunk i+1 to the device and the copy of chunk i-1 back run on two
    // streams of the handle beside the kernel of chunk i on the caller's stream.  The whole call
    // is ordered after earlier work on `stream`, and `stream` ends up waiting for the last copy.
    if (!h->pipe_ready) {
        CK(cudaStreamCreateWithFlags(&h->copy_in, cudaStreamNonBlocking));
        CK(cudaStreamCreateWithFlags(&h->copy_out, cudaStreamNonBlocking));
        CK(cudaEventCreateWithFlags(&h->ev_start, cudaEventDisableTiming));
        CK(cudaEventCreateWithFlags(&h->ev_done, cudaEventDisableTiming));
        for (int i = 0; i < dhq_handle_s::kHostChunks; ++i) {
            CK(cudaEventCreateWithFlags(&h->ev_in[i], cudaEventDisableTiming));
            CK(cudaEventCreateWithFlags(&h->ev_k[i], cudaEventDisableTiming));
        }
        h->pipe_ready = true;
    }
    CK(cudaEventRecord(h->ev_start, st));
    CK(cudaStreamWaitEvent(h->copy_in, h->ev_start, 0));
    CK(cudaStreamWaitEvent(h->copy_out, h->ev_start, 0));
    const int64_t base = rounds / chunks, extra = rounds % chunks;
    int64_t t0 = 0;
    for (int i = 0; i < chunks; ++i) {
        int64_t cnt = (base + (i < extra ? 1 : 0)) * round;
        if (cnt > n - t0) cnt = n - t0;
        CK(cudaMemcpyAsync(h->stage_in + t0 * 2, coords_host + t0 * 2, (size_t)cnt * 2 * sizeof(float),
                           cudaMemcpyHostToDevice, h->copy_in));
        CK(cudaEventRecord(h->ev_in[i], h->copy_in));
        CK(cudaStreamWaitEvent(st, h->ev_in[i], 0));
        dhq_status_t s = run_forward(h, h->stage_in + t0 * 2, cnt, h->stage_out + t0 * h->d_L, false, st);
        if (s != DHQ_OK) return s;
        CK(cudaEventRecord(h->ev_k[i], st));
        CK(cudaStreamWaitEvent(h->copy_out, h->ev_k[i], 0));
        CK(cudaMemcpyAsync(out_host + t0 * h->d_L, h->stage_out + t0 * h->d_L, (size_t)cnt * h->d_L * sizeof(float),
                           cudaMemcpyDeviceToHost, h->copy_out));
        t0 += cnt;
    }
    CK(cudaEventRecord(h->ev_done, h->copy_out));
    CK(cudaStreamWaitEvent(st, h->ev_done, 0));
    return DHQ_OK;
}

dhq_status_t dhq_export(dhq_handle_t h, void *host_buf, int64_t capacity, int64_t *needed)
{
    if (!h || !needed || capacity < 0) return DHQ_ERR_INVALID_ARG;
    if (!on_own_device(h)) return DHQ_ERR_INVALID_ARG;
    size_t payload = 0;
    for (int l = 0; l < h->L; ++l) {
        ArrayRef t[kLayerArrays];
        layer_arrays(h->layer[l], t);
        for (const ArrayRef &a : t) payload += a.bytes;
    }
    *needed = (int64_t)(sizeof(BlobHeader) + payload);
    if (!host_buf) return DHQ_OK;                       // size query
    if (capacity < *needed) return DHQ_ERR_TOO_LARGE;
    CK(cudaDeviceSynchronize());
    uint8_t *dst = static_cast<uint8_t *>(host_buf) + sizeof(BlobHeader);
    for (int l = 0; l < h->L; ++l) {
        ArrayRef t[kLayerArrays];
        layer_arrays(h->layer[l], t);
        for (const ArrayRef &a : t) {
            CK(cudaMemcpy(dst, *a.ptr, a.bytes, cudaMemcpyDeviceToHost));
            dst += a.bytes;
        }
    }
    BlobHeader hd;
    memset(&hd, 0, sizeof(hd));
    memcpy(hd.magic, kBlobMagic, 8);
    hd.version = kBlobVersion;
    hd.header_bytes = (uint32_t)sizeof(BlobHeader);
    hd.n_layers = h->L;
    for (int i = 0; i <= h->L; ++i) hd.dims[i] = h->dims[i];
    hd.w_bits = h->cfg.w_bits; hd.a_bits = h->cfg.a_bits;
    hd.w_gran = (int)h->cfg.w_gran; hd.a_gran = (int)h->cfg.a_gran; hd.rotation = (int)h->cfg.rotation;
    hd.omega0 = h->cfg.omega0;
    hd.activation = (int)h->cfg.activation; hd.act_s0 = h->cfg.act_s0;
    hd.calibrated = h->calibrated ? 1 : 0;
    hd.calib_layers_done = h->calib_layers_done;
    hd.has_fused = h->fused ? 1 : 0;
    for (int l = 0; l < h->L; ++l) {
        hd.epi_mode[l] = h->layer[l].epi_mode;
        hd.phase_bound[l] = h->layer[l].phase_bound;
    }
    hd.payload_bytes = payload;
    hd.payload_fnv1a = fnv1a(static_cast<uint8_t *>(host_buf) + sizeof(BlobHeader), payload);
    memcpy(host_buf, &hd, sizeof(hd));
    return DHQ_OK;
}

dhq_status_t dhq_import(const void *host_buf, int64_t bytes, void *stream, dhq_handle_t *out)
{
    if (!host_buf || !out || bytes < (int64_t)sizeof(BlobHeader)) return DHQ_ERR_INVALID_ARG;
    *out = nullptr;
    BlobHeader hd;
    memcpy(&hd, host_buf, sizeof(hd));
    if (memcmp(hd.magic, kBlobMagic, 8) != 0 || hd.version != kBlobVersion || hd.header_bytes != sizeof(BlobHeader))
        return DHQ_ERR_INVALID_ARG;
    if (hd.n_layers < 2 || hd.n_layers > kMaxLayers) return DHQ_ERR_INVALID_ARG;
    dhq_config_t cfg;
    int dims[kMaxLayers + 1];
    for (int i = 0; i <= hd.n_layers; ++i) dims[i] = hd.dims[i];
    cfg.n_layers = hd.n_layers; cfg.dims = dims;
    cfg.w_bits = hd.w_bits; cfg.a_bits = hd.a_bits; cfg.omega0 = hd.omega0;
    cfg.w_gran = (dhq_gran_t)hd.w_gran; cfg.a_gran = (dhq_gran_t)hd.a_gran; cfg.rotation = (dhq_rot_t)hd.rotation;
    cfg.activation = (dhq_act_t)hd.activation; cfg.act_s0 = hd.act_s0;
    dhq_status_t cs = check_config(&cfg);
    if (cs != DHQ_OK) return cs == DHQ_ERR_UNSUPPORTED ? DHQ_ERR_UNSUPPORTED : DHQ_ERR_INVALID_ARG;
    dhq_handle_s *h = new (std::nothrow) dhq_handle_s();
    if (!h) return DHQ_ERR_ALLOC;
    h->cfg = cfg;
    for (int i = 0; i <= hd.n_layers; ++i) h->dims[i] = dims[i];
    h->cfg.dims = h->dims;
    h->L = hd.n_layers; h->w = dims[1]; h->d_L = dims[hd.n_layers];
    h->float_mode = float_mode_of(cfg);
    h->gabor_s0 = cfg.activation == DHQ_ACT_GABOR ? (double)cfg.act_s0 : 0.0;
    size_t payload = 0;
    for (int l = 1; l <= h->L; ++l) {
        LayerDev &d = h->layer[l - 1];
        set_layer_dims(d, l, h->L, h->w, dims);
        d.has_f32 = h->float_mode == 2;
        d.has_uv = cfg.rotation == DHQ_ROT_BOTH && l == 1;
        ArrayRef t[kLayerArrays];
        layer_arrays(d, t);
        for (const ArrayRef &a : t) payload += a.bytes;
        const int e = hd.epi_mode[l - 1];
        if (e < EPI_LINEAR || e > EPI_SINE_MIXED) { delete h; return DHQ_ERR_INVALID_ARG; }
        d.epi_mode = e;
        d.phase_bound = hd.phase_bound[l - 1];
    }
    const uint8_t *src = static_cast<const uint8_t *>(host_buf) + sizeof(BlobHeader);
    if (hd.payload_bytes != payload || bytes < (int64_t)(sizeof(BlobHeader) + payload) || fnv1a(src, payload) != hd.payload_fnv1a) {
        delete h;
        return DHQ_ERR_INVALID_ARG;
    }
    cudaStream_t st = (cudaStream_t)stream;
    dhq_status_t rc = DHQ_OK;
    do {
        if (cudaGetDevice(&h->device) != cudaSuccess) { rc = DHQ_ERR_CUDA; break; }
        if (!dev_alloc(&h->d_status, 16)) { rc = DHQ_ERR_ALLOC; break; }
        if (cudaMemsetAsync(h->d_status, 0, 64, st) != cudaSuccess) { rc = DHQ_ERR_CUDA; break; }
        for (int l = 0; l < h->L && rc == DHQ_OK; ++l) {
            LayerDev &d = h->layer[l];
            if (!alloc_layer(d)) { rc = DHQ_ERR_ALLOC; break; }
            ArrayRef t[kLayerArrays];
            layer_arrays(d, t);
            for (const ArrayRef &a : t) {
                if (cudaMemcpyAsync(*a.ptr, src, a.bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) { rc = DHQ_ERR_CUDA; break; }
                src += a.bytes;
            }
        }
        if (rc != DHQ_OK) break;
        if (cudaStreamSynchronize(st) != cudaSuccess) { rc = DHQ_ERR_CUDA; break; } // host_buf may go after the call
        h->calibrated = hd.calibrated != 0;
        h->calib_layers_done = hd.calib_layers_done;
        if (hd.has_fused) rc = fused_create(h);
    } while (0);
    if (rc != DHQ_OK) {
        dhq_destroy(h);
        return rc;
    }
    *out = h;
    return DHQ_OK;
}

dhq_status_t dhq_layer_dims(dhq_handle_t h, int layer, int *K, int *M)
{
    if (!h || layer < 1 || layer > h->L) return DHQ_ERR_INVALID_ARG;
    if (K) *K = h->layer[layer - 1].K;
    if (M) *M = h->layer[layer - 1].M;
    return DHQ_OK;
}

dhq_status_t dhq_get_layer(dhq_handle_t h, int layer, int8_t *codes, float *w_scales, float *act_absmax)
{
    if (!h || layer < 1 || layer > h->L) return DHQ_ERR_INVALID_ARG;
    if (!on_own_device(h)) return DHQ_ERR_INVALID_ARG;
    const LayerDev &d = h->layer[layer - 1];
    CK(cudaDeviceSynchronize());
    if (codes) CK(cudaMemcpy(codes, d.qw, (size_t)d.M * d.K, cudaMemcpyDeviceToHost));
    if (w_scales) CK(cudaMemcpy(w_scales, d.s_w, (size_t)d.M * sizeof(float), cudaMemcpyDeviceToHost));
    if (act_absmax) {
        *act_absmax = NAN;
        if (h->cfg.a_gran == DHQ_GRAN_TENSOR && h->calibrated)
            CK(cudaMemcpy(act_absmax, d.act, sizeof(float), cudaMemcpyDeviceToHost));
    }
    return DHQ_OK;
}

dhq_status_t dhq_last_status(dhq_handle_t h)
{
    if (!h || !on_own_device(h)) return DHQ_ERR_INVALID_ARG;
    int v = 0;
    CK(cudaDeviceSynchronize());
    CK(cudaMemcpy(&v, h->d_status, sizeof(int), cudaMemcpyDeviceToHost));
    CK(cudaMemset(h->d_status, 0, sizeof(int)));
    return v == 0 ? DHQ_OK : DHQ_ERR_TIMEOUT;
}

dhq_status_t dhq_last_launch_clock(dhq_handle_t h, double *sm_mhz, double *milliseconds)
{
    if (!h || !on_own_device(h)) return DHQ_ERR_INVALID_ARG;
    if (!h->fused) return DHQ_ERR_UNSUPPORTED;
    long long words[5] = {0, 0, 0, 0, 0};
    CK(cudaDeviceSynchronize());
    CK(cudaMemcpy(words, h->d_status, sizeof(words), cudaMemcpyDeviceToHost));
    const double cycles = (double)(words[3] - words[1]), ns = (double)(words[4] - words[2]);
    if (!(ns > 0.0)) return DHQ_ERR_INVALID_ARG; // no fused launch yet
    if (sm_mhz) *sm_mhz = cycles / ns * 1e3;
    if (milliseconds) *milliseconds = ns * 1e-6;
    return DHQ_OK;
}

int64_t dhq_launch_count(dhq_handle_t h) { return h ? h->launches : 0; }

// Call log: with the environment variable DHQ_LOG set (to anything but "0") the main entry points
// write one line per call to stderr - the call, its size, the handle's shape, the status returned and
// the number of kernels it enqueued.  Read once per process; costs one predictable branch otherwise.
static bool log_enabled()
{
    static const bool on = [] {
        const char *v = getenv("DHQ_LOG");
        return v && v[0] && !(v[0] == '0' && !v[1]);
    }();
    return on;
}
static void log_call(const char *fn, dhq_handle_t h, int64_t n, int64_t launches_before, dhq_status_t s)
{
    if (!h) { fprintf(stderr, "[dhq] %s n=%lld -> %s\n", fn, (long long)n, dhq_status_string(s)); return; }
    fprintf(stderr, "[dhq] %s n=%lld (L=%d w=%d d_L=%d W%dA%d rot=%d gran=%d/%d%s) -> %s, %lld kernel(s)\n", fn, (long long)n,
            h->L, h->w, h->d_L, h->cfg.w_bits, h->cfg.a_bits, (int)h->cfg.rotation, (int)h->cfg.w_gran, (int)h->cfg.a_gran,
            h->fused ? ", fused" : ", layer by layer", dhq_status_string(s), (long long)(h->launches - launches_before));
}

dhq_status_t dhq_prepare(const dhq_config_t *cfg, const float *const *W, const float *const *b, void *stream, dhq_handle_t *out)
{
    const dhq_status_t s = prepare_impl(cfg, W, b, stream, out);
    if (log_enabled()) log_call("dhq_prepare", (s == DHQ_OK && out) ? *out : nullptr, 0, 0, s);
    return s;
}
dhq_status_t dhq_calibrate(dhq_handle_t h, const float *coords, int64_t n, void *stream)
{
    const int64_t before = h ? h->launches : 0;
    const dhq_status_t s = calibrate_entry(h, coords, n, stream);
    if (log_enabled()) log_call("dhq_calibrate", h, n, before, s);
    return s;
}
dhq_status_t dhq_forward(dhq_handle_t h, const float *coords, int64_t n, float *out, void *stream)
{
    if (!log_enabled()) return forward_entry(h, coords, n, out, stream);
    const int64_t before = h ? h->launches : 0;
    const dhq_status_t s = forward_entry(h, coords, n, out, stream);
    log_call("dhq_forward", h, n, before, s);
    return s;
}
dhq_status_t dhq_forward_host(dhq_handle_t h, const float *coords_host, int64_t n, float *out_host, void *stream)
{
    if (!log_enabled()) return forward_host_entry(h, coords_host, n, out_host, stream);
    const int64_t before = h ? h->launches : 0;
    const dhq_status_t s = forward_host_entry(h, coords_host, n, out_host, stream);
    log_call("dhq_forward_host", h, n, before, s);
    return s;
}

} // extern "C"
