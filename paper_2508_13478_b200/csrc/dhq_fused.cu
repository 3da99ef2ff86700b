// Fused forward kernel: the whole quantized INR (Sections III-B and III-C of the paper) for a
// tile of 128 coordinates without activations leaving the SM between layers.
//
// One persistent CTA per SM, 10 warps:
//   warps 0-3, 4-7  two epilogue groups; each owns a "slot": one tile of 128 tokens in flight,
//                   thread = one token (TMEM lane), so rotation, absmax and quantizer are
//                   thread-local and need no exchange between threads.
//   warp 8          issues tcgen05.mma kind::i8 (int8 x int8 -> int32 in tensor memory).
//   warp 9          brings the packed weight codes into shared memory with bulk async copies:
//                   once, if every hidden layer fits (they then stay resident), else through a
//                   ring that is refilled layer by layer from L2.
// While one slot's threads run their epilogue on the CUDA cores, the tensor core works on the
// other slot's tile.
//
// Per layer and tile:  acc (TMEM, int32) -> dequantize, bias, sine (dhq_math.cuh) -> fp32
//   -> butterfly stages with stride < 64 inside a 64-column register chunk -> the chunk goes back
//   to the same TMEM columns as fp32 -> the remaining stages (stride 64, 128) combine one value
//   from each chunk -> (per token: absmax, second trip through TMEM) -> quantize, pack 16 codes
//   -> st.shared into the next layer's A operand tile -> mbarrier -> next MMA.
// Layer 1 (K = 4) runs on the CUDA cores (one dp4a per output); the last layer is an MMA with
// N = 16 whose first d_L columns are the result.
//
// Every wait on an mbarrier is bounded: when it runs out the kernel records an error in the
// handle's status word, all roles leave their loops, tensor memory is released and the kernel
// returns.
#include <cstring>
#include <new>
#include "dhq_internal.cuh"
#include "dhq_tmem.cuh"

namespace dhq {

constexpr int kTile = 128;
constexpr int kThreads = 320;
constexpr int kMmaWarp = 8, kLoadWarp = 9;
constexpr int kMaxStages = 32;
constexpr unsigned long long kWaitLimitNs = 2000000000ull; // 2 s per wait
constexpr int kMinSmem = 120 * 1024; // more than half an SM's shared memory: one CTA per SM

struct FusedLayer {
    const uint8_t *qw_umma;
    const uint32_t *qw_k4m;
    const float *cA, *cA_lo, *cB;
    const float *act;
    int epi_mode;
    int pad_;
};

struct FusedParams {
    const float *coords;
    float *out;
    long long n, n_tiles;
    int L, W, d_L, per_token;
    float qmaxf;
    int n_stages, resident;
    int *status;
    FusedLayer layer[kMaxLayers];
};

struct FusedState {
    FusedParams p;
    size_t smem_bytes;
    int sm_count;
};

// Shared-memory map (offsets from a 1024-byte aligned base).
struct SmemMap {
    uint32_t a_tile[2];
    uint32_t ring;
    uint32_t last_w;
    uint32_t acc_full[2], codes_full[2], last_full, drain;
    uint32_t w_full, w_empty; // arrays of kMaxStages barriers
    uint32_t tmem_holder, abort_flag;
    uint32_t total;
};

__host__ __device__ inline SmemMap smem_map(int W, int n_stages)
{
    SmemMap m;
    uint32_t off = 0;
    m.a_tile[0] = off; off += kTile * W;
    m.a_tile[1] = off; off += kTile * W;
    m.ring = off; off += (uint32_t)n_stages * W * W;
    m.last_w = off; off += 16 * W;
    m.acc_full[0] = off; off += 8;
    m.acc_full[1] = off; off += 8;
    m.codes_full[0] = off; off += 8;
    m.codes_full[1] = off; off += 8;
    m.last_full = off; off += 8;
    m.drain = off; off += 8;
    m.w_full = off; off += 8 * kMaxStages;
    m.w_empty = off; off += 8 * kMaxStages;
    m.tmem_holder = off; off += 8;
    m.abort_flag = off; off += 8;
    m.total = off;
    return m;
}

// Bounded wait.  Returns false when the wait ran out or another role already gave up.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = ptx::globaltimer();
    for (uint32_t spin = 1;; ++spin) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if ((spin & 0xff) == 0) {
            if (*abort_flag) return false;
            if (ptx::globaltimer() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                atomicExch(status, 1);
                return false;
            }
        }
    }
}

// In-register butterfly stages with strides 1 .. N/2 on N values: pair (i, i+h) -> (a+b, a-b).
template <int N> __device__ __forceinline__ void fwht_local(float (&f)[N])
{
#pragma unroll
    for (int h = 1; h < N; h <<= 1) {
#pragma unroll
        for (int i = 0; i < N; ++i) {
            if ((i & h) == 0) {
                float a = f[i], b = f[i + h];
                f[i] = __fadd_rn(a, b);
                f[i + h] = __fsub_rn(a, b);
            }
        }
    }
}

// Round-half-even to an integer code held in the low byte: clamp, then add 1.5 * 2^23 (the sum
// rounds to the integer grid, ties to even, and its low mantissa bits are the two's complement
// code).  Same integer as __float2int_rn(clamp(v * inv)).
__device__ __forceinline__ uint32_t code_bits(float v, float inv, float qmaxf)
{
    float t = __fmul_rn(v, inv);
    t = fmaxf(fminf(t, qmaxf), -qmaxf);
    return __float_as_uint(__fadd_rn(t, 12582912.0f));
}
__device__ __forceinline__ uint32_t pack4(uint32_t b0, uint32_t b1, uint32_t b2, uint32_t b3)
{
    uint32_t lo = __byte_perm(b0, b1, 0x0040);
    uint32_t hi = __byte_perm(b2, b3, 0x0040);
    return __byte_perm(lo, hi, 0x5410);
}
// Quantize 16 consecutive-k values of this thread's token and store them as one 16-byte k-group
// of the A operand tile: byte offset (k/16) * 2048 + row * 16.
__device__ __forceinline__ void store_codes16(uint32_t a_tile, int row, int kgroup, const float *v, float inv, float qmaxf)
{
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
        w[j] = pack4(code_bits(v[4 * j], inv, qmaxf), code_bits(v[4 * j + 1], inv, qmaxf),
                     code_bits(v[4 * j + 2], inv, qmaxf), code_bits(v[4 * j + 3], inv, qmaxf));
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a_tile + kgroup * 2048 + row * 16),
                 "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
}

// Dequantize + bias + activation of 64 consecutive channels starting at m0.
template <bool PER_TOKEN, int MODE>
__device__ __forceinline__ void epilogue64_mode(const FusedLayer &ly, int m0, float s_x, const int (&acc)[64], float (&f)[64])
{
    const float4 *cA4 = reinterpret_cast<const float4 *>(ly.cA + m0);
    const float4 *cL4 = reinterpret_cast<const float4 *>(ly.cA_lo + m0);
    const float4 *cB4 = reinterpret_cast<const float4 *>(ly.cB + m0);
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        float4 a = __ldg(cA4 + j), b = __ldg(cB4 + j);
        float4 lo = make_float4(0.f, 0.f, 0.f, 0.f);
        if (MODE == EPI_SINE_WIDE) lo = __ldg(cL4 + j);
        const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w}, lv[4] = {lo.x, lo.y, lo.z, lo.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float c_hi = av[e], c_lo = lv[e];
            if (PER_TOKEN) token_const(av[e], lv[e], s_x, c_hi, c_lo);
            f[4 * j + e] = epilogue(MODE, (float)acc[4 * j + e], c_hi, c_lo, bv[e]);
        }
    }
}
template <bool PER_TOKEN>
__device__ __forceinline__ void epilogue64(const FusedLayer &ly, int m0, float s_x, const int (&acc)[64], float (&f)[64])
{
    if (ly.epi_mode == EPI_SINE_FAST) epilogue64_mode<PER_TOKEN, EPI_SINE_FAST>(ly, m0, s_x, acc, f);
    else epilogue64_mode<PER_TOKEN, EPI_SINE_WIDE>(ly, m0, s_x, acc, f);
}

// After the 64-column chunks have been through the local stages: the remaining stages, the
// quantizer and the store of the codes.  W = 64: everything is still in registers (f).
// W > 64: chunk c of the token sits in TMEM columns [c*64, c*64+64) as fp32.
// Returns the token's activation scale s_x of this layer (needed by the next epilogue).
template <int W, bool PER_TOKEN>
__device__ __forceinline__ float cross_and_quantize(uint32_t taddr, uint32_t a_tile, int row, float (&f)[64],
                                                    float static_s, float static_inv, float qmaxf)
{
    constexpr int NCH = W / 64;
    if constexpr (NCH == 1) {
        float s = static_s, inv = static_inv;
        if (PER_TOKEN) {
            float a = 0.f;
#pragma unroll
            for (int i = 0; i < 64; ++i) a = fmaxf(a, fabsf(f[i]));
            scales_of(a, qmaxf, s, inv);
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) store_codes16(a_tile, row, g, &f[16 * g], inv, qmaxf);
        return s;
    } else {
        constexpr int G = 64 / NCH; // local indices per group: NCH * G = 64 values in registers
        constexpr int NG = 64 / G;
        ptx::tmem_wait_st();
        float amax = 0.f;
#pragma unroll 1
        for (int g = 0; g < NG; ++g) {
            uint32_t u[NCH][G];
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                if constexpr (G == 16) ptx::tmem_ld16(taddr + c * 64 + g * G, u[c]);
                else if constexpr (G == 32) ptx::tmem_ld32(taddr + c * 64 + g * G, u[c]);
                else ptx::tmem_ld8(taddr + c * 64 + g * G, u[c]);
            }
            ptx::tmem_wait_ld();
            // strides 64, 128, ...: chunk index is the butterfly index
#pragma unroll
            for (int h = 1; h < NCH; h <<= 1) {
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    if ((c & h) == 0) {
#pragma unroll
                        for (int i = 0; i < G; ++i) {
                            float a = __uint_as_float(u[c][i]), b = __uint_as_float(u[c + h][i]);
                            u[c][i] = __float_as_uint(__fadd_rn(a, b));
                            u[c + h][i] = __float_as_uint(__fsub_rn(a, b));
                        }
                    }
                }
            }
            if (PER_TOKEN) {
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
#pragma unroll
                    for (int i = 0; i < G; ++i) amax = fmaxf(amax, fabsf(__uint_as_float(u[c][i])));
                    if constexpr (G == 16) ptx::tmem_st16(taddr + c * 64 + g * G, u[c]);
                    else if constexpr (G == 32) ptx::tmem_st32(taddr + c * 64 + g * G, u[c]);
                    else ptx::tmem_st8(taddr + c * 64 + g * G, u[c]);
                }
            } else {
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
#pragma unroll
                    for (int i = 0; i < G; i += 16) {
                        float v[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) v[e] = __uint_as_float(u[c][i + e]);
                        store_codes16(a_tile, row, (c * 64 + g * G + i) / 16, v, static_inv, qmaxf);
                    }
                }
            }
        }
        if (!PER_TOKEN) return static_s;
        float s, inv;
        scales_of(amax, qmaxf, s, inv);
        ptx::tmem_wait_st();
#pragma unroll 1
        for (int c = 0; c < NCH; ++c) {
            uint32_t u[64];
            ptx::tmem_ld64(taddr + c * 64, u);
            ptx::tmem_wait_ld();
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                float v[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) v[e] = __uint_as_float(u[16 * g + e]);
                store_codes16(a_tile, row, c * 4 + g, v, inv, qmaxf);
            }
        }
        return s;
    }
}

template <int W, bool PER_TOKEN>
__device__ void epilogue_role(const FusedParams &p, const SmemMap &sm, uint32_t smem_base, int slot, int quad, int lane,
                              uint32_t tmem_base, volatile int *abort_flag)
{
    constexpr int NCH = W / 64;
    const int row = quad * 32 + lane;
    const uint32_t taddr = tmem_base + (uint32_t)(slot * 256) + ((uint32_t)(quad * 32) << 16);
    const uint32_t a_tile = smem_base + sm.a_tile[slot];
    const uint32_t bar_acc = smem_base + sm.acc_full[slot], bar_codes = smem_base + sm.codes_full[slot];
    const float qmaxf = p.qmaxf;
    uint32_t acc_parity = 0;
    const FusedLayer &l1 = p.layer[0];

    for (long long r = 0;; ++r) {
        const long long tile = ((long long)blockIdx.x + r * gridDim.x) * 2 + slot;
        if (tile >= p.n_tiles) break;
        const long long tok = tile * kTile + row;
        const bool valid = tok < p.n;

        // ---------------- layer 1 on the CUDA cores: x~ = H_4 [x, y, 0, 0]
        float x = 0.f, y = 0.f;
        if (valid) {
            float2 c = __ldg(reinterpret_cast<const float2 *>(p.coords) + tok);
            x = c.x; y = c.y;
        }
        float r0 = __fadd_rn(x, y), r1 = __fsub_rn(x, y), r2 = __fadd_rn(0.f, 0.f), r3 = __fsub_rn(0.f, 0.f);
        float e0 = __fadd_rn(r0, r2), e2 = __fsub_rn(r0, r2), e1 = __fadd_rn(r1, r3), e3 = __fsub_rn(r1, r3);
        float s_x, inv_x;
        if (PER_TOKEN) {
            float a = fmaxf(fmaxf(fabsf(e0), fabsf(e1)), fmaxf(fabsf(e2), fabsf(e3)));
            scales_of(a, qmaxf, s_x, inv_x);
        } else {
            s_x = __ldg(l1.act + 1);
            inv_x = __ldg(l1.act + 2);
        }
        const uint32_t qx = pack4(code_bits(e0, inv_x, qmaxf), code_bits(e1, inv_x, qmaxf),
                                  code_bits(e2, inv_x, qmaxf), code_bits(e3, inv_x, qmaxf));
        float next_s = 1.f, next_inv = 0.f;
        if (!PER_TOKEN) {
            next_s = __ldg(p.layer[1].act + 1);
            next_inv = __ldg(p.layer[1].act + 2);
        }
        {
            float f[64];
#pragma unroll 1
            for (int ch = 0; ch < NCH; ++ch) {
                int acc[64];
                const uint4 *w4 = reinterpret_cast<const uint4 *>(l1.qw_k4m + ch * 64);
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    uint4 w = __ldg(w4 + j);
                    acc[4 * j + 0] = __dp4a((int)qx, (int)w.x, 0);
                    acc[4 * j + 1] = __dp4a((int)qx, (int)w.y, 0);
                    acc[4 * j + 2] = __dp4a((int)qx, (int)w.z, 0);
                    acc[4 * j + 3] = __dp4a((int)qx, (int)w.w, 0);
                }
                epilogue64_mode<PER_TOKEN, EPI_SINE_WIDE>(l1, ch * 64, s_x, acc, f);
                fwht_local<64>(f);
                if constexpr (NCH > 1) {
                    uint32_t u[64];
#pragma unroll
                    for (int i = 0; i < 64; ++i) u[i] = __float_as_uint(f[i]);
                    ptx::tmem_st64(taddr + ch * 64, u);
                }
            }
            s_x = cross_and_quantize<W, PER_TOKEN>(taddr, a_tile, row, f, next_s, next_inv, qmaxf);
        }
        ptx::fence_proxy_async();
        ptx::tc_fence_before();
        ptx::mbar_arrive(bar_codes);

        // ---------------- layers 2 .. L on the tensor core
        for (int l = 2; l <= p.L; ++l) {
            const FusedLayer &ly = p.layer[l - 1];
            if (!__all_sync(0xffffffffu, wait_bar(bar_acc, acc_parity, abort_flag, p.status))) return;
            acc_parity ^= 1;
            ptx::tc_fence_after();
            if (l < p.L) {
                if (!PER_TOKEN) {
                    next_s = __ldg(p.layer[l].act + 1);
                    next_inv = __ldg(p.layer[l].act + 2);
                }
                float f[64];
#pragma unroll 1
                for (int ch = 0; ch < NCH; ++ch) {
                    uint32_t u[64];
                    ptx::tmem_ld64(taddr + ch * 64, u);
                    ptx::tmem_wait_ld();
                    int acc[64];
#pragma unroll
                    for (int i = 0; i < 64; ++i) acc[i] = (int)u[i];
                    epilogue64<PER_TOKEN>(ly, ch * 64, s_x, acc, f);
                    fwht_local<64>(f);
                    if constexpr (NCH > 1) {
#pragma unroll
                        for (int i = 0; i < 64; ++i) u[i] = __float_as_uint(f[i]);
                        ptx::tmem_st64(taddr + ch * 64, u);
                    }
                }
                s_x = cross_and_quantize<W, PER_TOKEN>(taddr, a_tile, row, f, next_s, next_inv, qmaxf);
                ptx::fence_proxy_async();
                ptx::tc_fence_before();
                ptx::mbar_arrive(bar_codes);
            } else {
                uint32_t u[4];
                ptx::tmem_ld4(taddr, u);
                ptx::tmem_wait_ld();
                ptx::tc_fence_before();
                if (valid) {
#pragma unroll
                    for (int m = 0; m < 4; ++m) {
                        if (m < p.d_L) {
                            float c_hi = __ldg(ly.cA + m), c_lo = 0.f;
                            if (PER_TOKEN) c_hi = __fmul_rn(c_hi, s_x);
                            p.out[tok * p.d_L + m] = epilogue(EPI_LINEAR, (float)(int)u[m], c_hi, c_lo, __ldg(ly.cB + m));
                        }
                    }
                }
            }
        }
    }
}

template <int W>
__device__ void mma_role(const FusedParams &p, const SmemMap &sm, uint32_t smem_base, uint32_t tmem_base,
                         volatile int *abort_flag)
{
    uint32_t codes_parity[2] = {0, 0};
    const uint32_t idesc_hidden = ptx::idesc_i8(kTile, W), idesc_last = ptx::idesc_i8(kTile, 16);
    long long use = 0; // ring uses so far (streaming mode)
    bool ok = true;
    for (long long r = 0; ok; ++r) {
        const long long tile0 = ((long long)blockIdx.x + r * gridDim.x) * 2;
        if (tile0 >= p.n_tiles) break;
        const bool active1 = tile0 + 1 < p.n_tiles;
        for (int l = 2; l <= p.L && ok; ++l) {
            uint32_t b_addr, n_rows, idesc;
            int stage = 0;
            if (l < p.L) {
                stage = p.resident ? (l - 2) : (int)(use % p.n_stages);
                uint32_t par = p.resident ? 0u : (uint32_t)((use / p.n_stages) & 1);
                if (!wait_bar(smem_base + sm.w_full + 8 * stage, par, abort_flag, p.status)) { ok = false; break; }
                b_addr = smem_base + sm.ring + (uint32_t)stage * W * W;
                n_rows = W;
                idesc = idesc_hidden;
            } else {
                if (!wait_bar(smem_base + sm.last_full, 0, abort_flag, p.status)) { ok = false; break; }
                b_addr = smem_base + sm.last_w;
                n_rows = 16;
                idesc = idesc_last;
            }
            for (int s = 0; s < 2; ++s) {
                if (s == 1 && !active1) break;
                if (!wait_bar(smem_base + sm.codes_full[s], codes_parity[s], abort_flag, p.status)) { ok = false; break; }
                codes_parity[s] ^= 1;
                ptx::tc_fence_after();
                const uint32_t a_addr = smem_base + sm.a_tile[s];
                const uint32_t d = tmem_base + (uint32_t)(s * 256);
#pragma unroll 1
                for (int ks = 0; ks < W / 32; ++ks) {
                    uint64_t ad = ptx::smem_desc(a_addr + ks * 2 * (kTile * 16), kTile * 16, 128);
                    uint64_t bd = ptx::smem_desc(b_addr + ks * 2 * (n_rows * 16), n_rows * 16, 128);
                    ptx::mma_i8(d, ad, bd, idesc, ks > 0 ? 1u : 0u);
                }
                ptx::mma_commit(smem_base + sm.acc_full[s]);
            }
            if (!ok) break;
            if (l < p.L && !p.resident) {
                ptx::mma_commit(smem_base + sm.w_empty + 8 * stage);
                ++use;
            }
        }
    }
    if (!ok) { // give the MMAs already issued a bounded time to finish before TMEM is released
        ptx::mma_commit(smem_base + sm.drain);
        const unsigned long long t0 = ptx::globaltimer();
        while (!ptx::mbar_try_wait(smem_base + sm.drain, 0) && ptx::globaltimer() - t0 < kWaitLimitNs) {}
    }
}

template <int W>
__device__ void load_role(const FusedParams &p, const SmemMap &sm, uint32_t smem_base, volatile int *abort_flag)
{
    const uint32_t slab = W * W;
    ptx::mbar_expect_tx(smem_base + sm.last_full, 16 * W);
    ptx::bulk_g2s(smem_base + sm.last_w, p.layer[p.L - 1].qw_umma, 16 * W, smem_base + sm.last_full);
    const int hidden = p.L - 2;
    if (hidden <= 0) return;
    long long rounds = 0;
    for (long long r = 0;; ++r) {
        if (((long long)blockIdx.x + r * gridDim.x) * 2 >= p.n_tiles) break;
        ++rounds;
    }
    const long long total = p.resident ? hidden : rounds * hidden;
    long long issued = 0;
    bool ok = true;
    for (long long i = 0; i < total; ++i) {
        const int stage = (int)(i % p.n_stages);
        if (i >= p.n_stages) {
            uint32_t par = (uint32_t)(((i / p.n_stages) - 1) & 1);
            if (!wait_bar(smem_base + sm.w_empty + 8 * stage, par, abort_flag, p.status)) { ok = false; break; }
        }
        const int l = 2 + (int)(i % hidden);
        ptx::mbar_expect_tx(smem_base + sm.w_full + 8 * stage, slab);
        ptx::bulk_g2s(smem_base + sm.ring + (uint32_t)stage * slab, p.layer[l - 1].qw_umma, slab,
                      smem_base + sm.w_full + 8 * stage);
        ++issued;
    }
    if (!ok || *abort_flag) { // let copies in flight land before the CTA may exit
        const unsigned long long t0 = ptx::globaltimer();
        for (long long i = issued > p.n_stages ? issued - p.n_stages : 0; i < issued; ++i) {
            const int stage = (int)(i % p.n_stages);
            const uint32_t par = (uint32_t)((i / p.n_stages) & 1);
            while (!ptx::mbar_try_wait(smem_base + sm.w_full + 8 * stage, par) &&
                   ptx::globaltimer() - t0 < kWaitLimitNs) {}
        }
    }
}

template <int W, bool PER_TOKEN>
__global__ void __launch_bounds__(kThreads, 1) fused_kernel(const __grid_constant__ FusedParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t smem_base = (raw + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - raw);
    const SmemMap sm = smem_map(W, p.n_stages);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_gen + sm.abort_flag);
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(smem_gen + sm.tmem_holder);

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(smem_base + sm.acc_full[s], 1);
            ptx::mbar_init(smem_base + sm.codes_full[s], kTile);
        }
        ptx::mbar_init(smem_base + sm.last_full, 1);
        ptx::mbar_init(smem_base + sm.drain, 1);
        for (int i = 0; i < kMaxStages; ++i) {
            ptx::mbar_init(smem_base + sm.w_full + 8 * i, 1);
            ptx::mbar_init(smem_base + sm.w_empty + 8 * i, 1);
        }
        ptx::fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        ptx::tmem_alloc(smem_base + sm.tmem_holder, 512);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    if (warp < 8) {
        epilogue_role<W, PER_TOKEN>(p, sm, smem_base, warp >> 2, warp & 3, lane, tmem_base, abort_flag);
    } else if (warp == kMmaWarp) {
        if (lane == 0) mma_role<W>(p, sm, smem_base, tmem_base, abort_flag);
    } else {
        if (lane == 0) load_role<W>(p, sm, smem_base, abort_flag);
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        __syncwarp();
        ptx::tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------ host

typedef void (*fused_fn)(const FusedParams);

static fused_fn pick_kernel(int W, bool per_token)
{
    switch (W) {
    case 64: return per_token ? fused_kernel<64, true> : fused_kernel<64, false>;
    case 128: return per_token ? fused_kernel<128, true> : fused_kernel<128, false>;
    case 256: return per_token ? fused_kernel<256, true> : fused_kernel<256, false>;
    }
    return nullptr;
}

dhq_status_t fused_create(dhq_handle_s *h)
{
    FusedState *fs = new (std::nothrow) FusedState();
    if (!fs) return DHQ_ERR_ALLOC;
    memset(fs, 0, sizeof(*fs));
    h->fused = fs;
    FusedParams &p = fs->p;
    p.L = h->L; p.W = h->w; p.d_L = h->d_L;
    p.per_token = h->cfg.a_gran == DHQ_GRAN_CHANNEL_OR_TOKEN;
    p.qmaxf = (float)((1 << (h->cfg.a_bits - 1)) - 1);
    p.status = h->d_status;
    for (int l = 0; l < h->L; ++l) {
        const LayerDev &d = h->layer[l];
        p.layer[l].qw_umma = d.qw_umma;
        p.layer[l].qw_k4m = d.qw_k4m;
        p.layer[l].cA = d.cA; p.layer[l].cA_lo = d.cA_lo; p.layer[l].cB = d.cB;
        p.layer[l].act = d.act;
        p.layer[l].epi_mode = d.epi_mode;
    }
    fused_fn fn = pick_kernel(h->w, p.per_token);
    if (!fn) return DHQ_ERR_UNSUPPORTED;
    int dev = 0, max_optin = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&max_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&fs->sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return DHQ_ERR_CUDA;
    // weight ring: as many W*W stages as fit beside the two A tiles; all hidden layers resident
    // if they fit
    const int hidden = h->L - 2;
    const size_t fixed = smem_map(h->w, 0).total + 1024;
    int stages = (int)(((size_t)max_optin - fixed) / ((size_t)h->w * h->w));
    if (stages > kMaxStages) stages = kMaxStages;
    if (hidden > 0 && stages < 1) return DHQ_ERR_UNSUPPORTED;
    if (stages >= hidden) { p.resident = 1; p.n_stages = hidden > 0 ? hidden : 0; }
    else { p.resident = 0; p.n_stages = stages; }
    size_t bytes = smem_map(h->w, p.n_stages).total + 1024;
    if (bytes < (size_t)kMinSmem) bytes = kMinSmem;
    fs->smem_bytes = bytes;
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess)
        return DHQ_ERR_CUDA;
    return DHQ_OK;
}

void fused_destroy(dhq_handle_s *h)
{
    delete static_cast<FusedState *>(h->fused);
    h->fused = nullptr;
}

dhq_status_t fused_forward(dhq_handle_s *h, const float *coords, int64_t n, float *out, cudaStream_t st)
{
    FusedState *fs = static_cast<FusedState *>(h->fused);
    if (!fs) return DHQ_ERR_INVALID_ARG;
    FusedParams p = fs->p;
    p.coords = coords; p.out = out; p.n = n;
    p.n_tiles = (n + kTile - 1) / kTile;
    fused_fn fn = pick_kernel(h->w, p.per_token);
    long long pairs = (p.n_tiles + 1) / 2;
    int grid = (int)(pairs < fs->sm_count ? pairs : fs->sm_count);
    fn<<<grid, kThreads, fs->smem_bytes, st>>>(p);
    h->launches++;
    return cudaGetLastError() == cudaSuccess ? DHQ_OK : DHQ_ERR_CUDA;
}

} // namespace dhq
