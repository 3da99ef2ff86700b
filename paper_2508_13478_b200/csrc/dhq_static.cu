// dhq_forward_static_scratch: the layer-by-layer forward for callers that may not allocate
// device memory (see include/dhq.h).  Same kernel as the debug path (launch_layer); the
// activations between layers go through the fixed array below instead of buffers obtained from
// cudaMalloc.
#include <cstring>
#include <mutex>
#include "dhq_internal.cuh"

namespace {

constexpr int kMaxWidth = 512;
constexpr int kMaxDevices = 64;
constexpr size_t kHalf = (size_t)DHQ_STATIC_MAX_TOKENS * kMaxWidth; // floats per ping-pong half

// Part of the library image: present on every GPU that loads the library, 16 MiB.
static __device__ __align__(256) float g_static_scratch[2 * kHalf];

// In host code `g_static_scratch` is only a stand-in for the symbol; the address a kernel can
// use has to be asked for, per device.
float *g_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_setup_mutex;

dhq_status_t scratch_for_current_device(float **ptr)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DHQ_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        float *p = nullptr;
        if (cudaGetSymbolAddress((void **)&p, g_static_scratch) != cudaSuccess || !p) return DHQ_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *ptr = g_scratch_addr[dev];
    return DHQ_OK;
}

} // namespace

extern "C" dhq_status_t dhq_forward_static_scratch(dhq_handle_t h, const float *coords, int64_t n, float *out,
                                                   void *stream)
{
    using namespace dhq;
    if (!h || n < 0 || (n > 0 && (!coords || !out))) return DHQ_ERR_INVALID_ARG;
    if (!on_own_device(h)) return DHQ_ERR_INVALID_ARG; // the handle's buffers live on another GPU
    if (n > DHQ_STATIC_MAX_TOKENS) return DHQ_ERR_TOO_LARGE;
    if (n == 0) return DHQ_OK;
    if (h->w > kMaxWidth || h->cfg.rotation == DHQ_ROT_BOTH || h->float_mode || h->gabor_s0 > 0.0) return DHQ_ERR_UNSUPPORTED;
    if (!h->calibrated) return DHQ_ERR_NOT_CALIBRATED;
    float *scratch = nullptr;
    dhq_status_t s = scratch_for_current_device(&scratch);
    if (s != DHQ_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    const float *X = nullptr;
    for (int l = 1; l <= h->L; ++l) {
        const LayerDev &d = h->layer[l - 1];
        LayerArgs a;
        memset(&a, 0, sizeof(a));
        a.X = X; a.coords = coords; a.n = n;
        a.K = d.K; a.M = d.M; a.d_L = h->d_L;
        a.a_bits = h->cfg.a_bits;
        a.per_token = h->cfg.a_gran == DHQ_GRAN_CHANNEL_OR_TOKEN;
        a.epi_mode = d.epi_mode;
        a.rotate = h->cfg.rotation == DHQ_ROT_INPUT;
        a.qw_k4m = d.qw_k4m; a.cA = d.cA; a.cA_lo = d.cA_lo; a.cB = d.cB; a.act = d.act;
        a.fxP = d.fxP; a.fxQ = d.fxQ; a.fxB = d.fxB;
        a.Y = scratch + (size_t)((l - 1) & 1) * kHalf; // every row < n is written before it is read
        if (l == h->L) a.out = out;
        if (launch_layer(a, st) != cudaSuccess) return DHQ_ERR_CUDA;
        h->launches++;
        X = a.Y;
    }
    return DHQ_OK;
}
