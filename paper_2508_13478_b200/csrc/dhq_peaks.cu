// Micro-benchmarks of the pipes that bound the fused kernel (see include/dhq_peaks.h).
#include <cuda_runtime.h>
#include <cstring>
#include "../../include/dhq_peaks.h"
#include "dhq_internal.cuh"
#include "dhq_tmem.cuh"

namespace dhq {

constexpr int kChains = 8;

template <int PIPE> __global__ void __launch_bounds__(256) scalar_pipe_kernel(int iters, float seed, float *sink)
{
    float v[kChains];
    uint32_t u[kChains];
    unsigned long long w[kChains], k2;
    asm("mov.b64 %0, {%1, %1};" : "=l"(k2) : "f"(seed * 1e-3f));
#pragma unroll
    for (int c = 0; c < kChains; ++c) {
        v[c] = seed + (float)(threadIdx.x + c) * 1e-3f;
        u[c] = threadIdx.x * 2654435761u + c;
        asm("mov.b64 %0, {%1, %2};" : "=l"(w[c]) : "f"(v[c]), "f"(seed));
    }
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int rep = 0; rep < 8; ++rep) {
#pragma unroll
            for (int c = 0; c < kChains; ++c) {
                if (PIPE == DHQ_PIPE_FFMA) v[c] = __fmaf_rn(v[c], 0.999f, 1e-3f);
                else if (PIPE == DHQ_PIPE_FADD) v[c] = __fadd_rn(v[c], 1e-3f);
                else if (PIPE == DHQ_PIPE_MUFU_SIN) asm volatile("sin.approx.f32 %0, %0;" : "+f"(v[c]));
                else if (PIPE == DHQ_PIPE_I2F) asm volatile("cvt.rn.f32.s32 %0, %1;" : "=f"(v[c]) : "r"(u[c] ^ __float_as_uint(v[c])));
                else if (PIPE == DHQ_PIPE_F2I) asm volatile("cvt.rni.s32.f32 %0, %1;" : "=r"(u[c]) : "f"(__uint_as_float((u[c] & 0x007fffffu) | 0x3f800000u)));
                else if (PIPE == DHQ_PIPE_PRMT) asm volatile("prmt.b32 %0, %0, %1, 0x5140;" : "+r"(u[c]) : "r"(u[(c + 1) % kChains]));
                else if (PIPE == DHQ_PIPE_FMNMX) v[c] = fmaxf(fminf(v[c], seed), -seed);
                else if (PIPE == DHQ_PIPE_FADD2) asm volatile("add.rn.f32x2 %0, %0, %1;" : "+l"(w[c]) : "l"(k2));
                else if (PIPE == DHQ_PIPE_FFMA2) asm volatile("fma.rn.f32x2 %0, %0, %1, %1;" : "+l"(w[c]) : "l"(k2));
            }
        }
    }
    float acc = 0.f;
#pragma unroll
    for (int c = 0; c < kChains; ++c) acc += v[c] + __uint_as_float(u[c] & 0x3fffffffu) + __uint_as_float((uint32_t)(w[c] >> 32) & 0x3fffffffu);
    if (acc == 123.456f) sink[0] = acc; // keeps the loop alive
}

// One CTA per SM: A (128 x 256 B) and B (256 x 256 B) zero-filled in shared memory, then `iters`
// groups of 8 MMAs (K = 8 * 32) into alternating halves of tensor memory.
__global__ void __launch_bounds__(128) tensor_i8_kernel(int iters, int *status)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - raw);
    const uint32_t a_off = 0, b_off = 128 * 256, bar_off = b_off + 256 * 256, holder_off = bar_off + 8;
    for (uint32_t i = threadIdx.x; i < (bar_off >> 2); i += blockDim.x) reinterpret_cast<uint32_t *>(gen)[i] = 0;
    if (threadIdx.x == 0) {
        ptx::mbar_init(base + bar_off, 1);
        ptx::fence_mbar_init();
    }
    if (threadIdx.x < 32) {
        ptx::tmem_alloc(base + holder_off, 512);
        ptx::tmem_relinquish();
    }
    ptx::fence_proxy_async();
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(gen + holder_off);
    if (threadIdx.x == 0) {
        const uint32_t idesc = ptx::idesc_i8(128, 256);
        uint32_t parity = 0;
        bool ok = true;
        for (int it = 0; it < iters && ok; it += 16) {
            for (int j = 0; j < 16 && it + j < iters; ++j) {
                const uint32_t d = tmem + (uint32_t)(((it + j) & 1) * 256);
#pragma unroll 1
                for (int ks = 0; ks < 8; ++ks) {
                    uint64_t ad = ptx::smem_desc(base + a_off + ks * 2 * 2048, 2048, 128);
                    uint64_t bd = ptx::smem_desc(base + b_off + ks * 2 * 4096, 4096, 128);
                    ptx::mma_i8(d, ad, bd, idesc, ks > 0 ? 1u : 0u);
                }
            }
            ptx::mma_commit(base + bar_off);
            const unsigned long long t0 = ptx::globaltimer();
            while (!ptx::mbar_try_wait(base + bar_off, parity)) {
                if (ptx::globaltimer() - t0 > 1000000000ull) { ok = false; atomicExch(status, 1); break; }
            }
            parity ^= 1;
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) ptx::tmem_dealloc(tmem, 512);
}

template <int PIPE> static cudaError_t run_scalar(int blocks, int iters, float *sink, cudaStream_t st)
{
    scalar_pipe_kernel<PIPE><<<blocks, 256, 0, st>>>(iters, 1.5f, sink);
    return cudaGetLastError();
}

// Largest |f(x) - sin(x)| over `count` fp32 arguments spread evenly over [lo, hi]; f is the
// hardware approximation alone (mode 0) or with the explicit 2 pi reduction in front (mode 1); the
// reference is the fp64 sine of the same fp32 argument.
__global__ void sine_error_kernel(float lo, float hi, long long count, int mode, unsigned long long *worst_bits)
{
    double worst = 0.0;
    const double step = count > 1 ? ((double)hi - (double)lo) / (double)(count - 1) : 0.0;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x) {
        const float x = (float)((double)lo + step * (double)i);
        const float y = mode == 1 ? sin_wide(x) : sin_approx(x);
        const double e = fabs((double)y - sin((double)x));
        if (e > worst) worst = e;
    }
    atomicMax(worst_bits, (unsigned long long)__double_as_longlong(worst)); // non-negative doubles order as integers
}

} // namespace dhq

extern "C" int dhq_measure_sine_error(float lo, float hi, long long count, int mode, void *stream, double *max_abs_err)
{
    if (!max_abs_err || count < 1 || !(lo <= hi) || (mode != 0 && mode != 1)) return -1;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned long long *d = nullptr, bits = 0;
    if (cudaMalloc(&d, sizeof(bits)) != cudaSuccess) return -3;
    int rc = 0;
    if (cudaMemsetAsync(d, 0, sizeof(bits), st) != cudaSuccess) rc = -5;
    if (rc == 0) {
        dhq::sine_error_kernel<<<1024, 256, 0, st>>>(lo, hi, count, mode, d);
        if (cudaGetLastError() != cudaSuccess || cudaMemcpyAsync(&bits, d, sizeof(bits), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess)
            rc = -6;
    }
    cudaFree(d);
    if (rc == 0) memcpy(max_abs_err, &bits, sizeof(double));
    return rc;
}

extern "C" int dhq_measure_pipe(int pipe, int iters, void *stream, double *ops_per_s, double *ms)
{
    using namespace dhq;
    if (!ops_per_s || iters < 1) return -1;
    cudaStream_t st = (cudaStream_t)stream;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -2;
    float *sink = nullptr;
    if (cudaMalloc(&sink, 256) != cudaSuccess) return -3;
    cudaMemset(sink, 0, 256);
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    const int blocks = sms * 8;
    const size_t tensor_smem = 128 * 256 + 256 * 256 + 64 + 1024;
    int rc = 0;
    float t = 0.f;
    for (int rep = 0; rep < 2 && rc == 0; ++rep) {
        cudaEventRecord(e0, st);
        cudaError_t e = cudaSuccess;
        switch (pipe) {
        case DHQ_PIPE_FFMA: e = run_scalar<DHQ_PIPE_FFMA>(blocks, iters, sink, st); break;
        case DHQ_PIPE_FADD: e = run_scalar<DHQ_PIPE_FADD>(blocks, iters, sink, st); break;
        case DHQ_PIPE_MUFU_SIN: e = run_scalar<DHQ_PIPE_MUFU_SIN>(blocks, iters, sink, st); break;
        case DHQ_PIPE_I2F: e = run_scalar<DHQ_PIPE_I2F>(blocks, iters, sink, st); break;
        case DHQ_PIPE_F2I: e = run_scalar<DHQ_PIPE_F2I>(blocks, iters, sink, st); break;
        case DHQ_PIPE_PRMT: e = run_scalar<DHQ_PIPE_PRMT>(blocks, iters, sink, st); break;
        case DHQ_PIPE_FMNMX: e = run_scalar<DHQ_PIPE_FMNMX>(blocks, iters, sink, st); break;
        case DHQ_PIPE_FADD2: e = run_scalar<DHQ_PIPE_FADD2>(blocks, iters, sink, st); break;
        case DHQ_PIPE_FFMA2: e = run_scalar<DHQ_PIPE_FFMA2>(blocks, iters, sink, st); break;
        case DHQ_PIPE_TENSOR_I8:
            e = cudaFuncSetAttribute(tensor_i8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tensor_smem);
            if (e == cudaSuccess) {
                tensor_i8_kernel<<<sms, 128, tensor_smem, st>>>(iters, (int *)sink);
                e = cudaGetLastError();
            }
            break;
        case DHQ_PIPE_PASS1: e = launch_pass_rate(1, sms, iters, st); break;
        case DHQ_PIPE_PASS2: e = launch_pass_rate(2, sms, iters, st); break;
        case DHQ_PIPE_PASS12: e = launch_pass_rate(3, sms, iters, st); break;
        default: rc = -4;
        }
        if (e != cudaSuccess) rc = -5;
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess) rc = -6;
        if (rc == 0) cudaEventElapsedTime(&t, e0, e1);
    }
    if (rc == 0) {
        double ops;
        if (pipe == DHQ_PIPE_TENSOR_I8) {
            int flag = 0;
            cudaMemcpy(&flag, sink, sizeof(int), cudaMemcpyDeviceToHost);
            if (flag) rc = 1;
            ops = (double)sms * iters * 8.0 * 2.0 * 128 * 256 * 32;
        } else if (pipe == DHQ_PIPE_PASS1 || pipe == DHQ_PIPE_PASS2 || pipe == DHQ_PIPE_PASS12) {
            ops = (double)sms * iters * 256.0 * 256.0; // activation elements: two tiles of 128 tokens x 256 per SM and iteration
        } else {
            double per_thread = (double)iters * 8 * kChains * ((pipe == DHQ_PIPE_FMNMX || pipe == DHQ_PIPE_FADD2 || pipe == DHQ_PIPE_FFMA2) ? 2 : 1);
            ops = per_thread * 256.0 * blocks;
        }
        *ops_per_s = ops / ((double)t * 1e-3);
        if (ms) *ms = t;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(sink);
    return rc;
}
