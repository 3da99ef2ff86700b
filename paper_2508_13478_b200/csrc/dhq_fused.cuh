// Fused forward kernel: the whole quantized INR (Sections III-B and III-C of the paper) for
// tiles of 128 coordinates without activations leaving the SM between layers.
//
// One persistent CTA per SM, 18 warps (19 at width 512):
//   warps 0-15  epilogue warps.  Width <= 256: two "slots" of 8 warps, each slot has one tile of
//               128 tokens in flight (its own A operand tile and 256 tensor-memory columns), so
//               that one slot's CUDA-core work overlaps the other slot's MMA; the second slot
//               starts half a layer period late.  Width 512: one slot of 16 warps; a layer's
//               weights arrive as eight pieces (256 output columns x 128 k, the first half of the
//               columns first), each feeding N = 256 MMAs; a thread has one chunk in each half
//               and starts on the first while the second half's weights and MMAs are under way.
//               A token (row) is a tensor-memory lane; R = 2 (or 4) threads from different warps
//               share a row and split its columns.
//   warp 16     issues tcgen05.mma kind::i8 (int8 x int8 -> int32 in tensor memory).
//   warp 18     (width 512) brings each tile's coordinates into shared memory with one bulk copy,
//               a tile ahead.
//   warp 17     brings the packed weight codes into shared memory with bulk async copies: once,
//               if every hidden layer fits (they then stay resident), else through a ring that
//               is refilled slab by slab from L2.
//
// Per layer and tile:
//   pass 1  each thread takes its chunks of 64 columns: acc (TMEM, int32) -> dequantize, bias,
//           sine (dhq_math.cuh) -> butterfly stages with stride < 64 in registers -> fp32 back to
//           the same TMEM columns.          [mbarrier of the R warps that share the 32 rows]
//   pass 2  each thread takes its groups: one value from every chunk at G consecutive positions
//           -> the remaining butterfly stages (stride 64, 128, ...) -> quantize, pack, st.shared
//           into the next layer's A operand tile -> mbarrier -> next MMA.
//           Per-token scales: the rotated values go back to TMEM once more while the row's
//           absmax is combined through shared memory, then pass 3 quantizes.
// Layer 1 (K = 4) runs on the CUDA cores; the last layer is an MMA with N = 16 whose first d_L
// columns are the result.
//
// Every wait on an mbarrier is bounded: when it runs out the kernel records an error in the
// handle's status word, all roles leave their loops, tensor memory is released and the kernel
// returns.
#pragma once
#include <cstring>
#include <new>
#include <type_traits>
#include "dhq_internal.cuh"
#include "dhq_tmem.cuh"

namespace dhq {

constexpr int kTile = 128;
constexpr int kEpiWarps = 16;
constexpr int kMmaWarp = 16, kLoadWarp = 17, kXyWarp = 18;
constexpr int kThreads = 18 * 32; // width 512 runs one more warp (Cfg::THREADS)
constexpr int kMaxStages = 32;
constexpr uint32_t kCopyBytes = 8192; // bytes per bulk copy of a weight slab
constexpr int kMinSmem = 120 * 1024; // more than half an SM's shared memory: one CTA per SM

// Work split for a hidden width W.
template <int W> struct Cfg {
    static constexpr int SLOTS = (W == 512) ? 1 : 2;
    static constexpr int R = kEpiWarps / (4 * SLOTS);          // threads per row: 2 or 4
    static constexpr int CH = (W == 64) ? 32 : 64;             // columns per register chunk (= fused_chunk(W))
    static constexpr int NCH = W / CH;                         // chunks per row
    static constexpr int CPT = NCH / R;                        // chunks per thread
    static constexpr int G = (64 / NCH < CH / R) ? 64 / NCH : CH / R; // positions per pass-2 group
    static constexpr int GPT = CH / (G * R);                   // groups per thread
    static constexpr int KSLABS = (W == 512) ? 4 : 1;          // weight slabs per layer along K
    static constexpr int SLABK = W / KSLABS;                   // k per slab (= fused_slab_k)
    static constexpr int NHALF = (W == 512) ? 2 : 1;           // MMAs along N (an MMA has N <= 256)
    static constexpr int NW = W / NHALF;                       // N of one MMA
    static constexpr int PIECES = KSLABS * NHALF;              // weight pieces per layer (ring units)
    static constexpr int PIECE_BYTES = SLABK * NW;             // 64 KB (width 256), 32 KB (width 512)
    static constexpr int SLOT_THREADS = R * kTile;
    // Width 512: the coordinates of a whole tile arrive by one bulk copy issued by a 19th warp (measured:
    // 2.6 % faster, 6.7 % from mapped host memory; narrower networks lost 4-7 % to the extra barrier).
    static constexpr bool BULK_XY = (W == 512);
    static constexpr int THREADS = kThreads + (BULK_XY ? 32 : 0);
    static constexpr int TMEM_COLS_PER_SLOT = 512 / SLOTS;
};

// Tile of slot `slot` of this CTA in its round r.  Normally the slots of a CTA take adjacent tiles.
// A launch with fewer tiles than CTAs x slots is spread instead: the tiles go round-robin first
// over the CTAs, then over the slots, so that it covers as many SMs as it has tiles (one busy slot
// each) before any SM gets a second tile.
template <bool SPREAD> __device__ __forceinline__ long long tile_index(long long r, int slot, int slots)
{
    return SPREAD ? (r * slots + slot) * (long long)gridDim.x + blockIdx.x
                  : ((long long)blockIdx.x + r * gridDim.x) * slots + slot;
}

// Chunk cc of the thread with index `sub` among the R threads of a row.  Width 512 gives every
// thread one chunk in each half of the columns (the halves' accumulators complete one after the
// other); otherwise a thread's chunks are adjacent.
template <int W> __device__ __forceinline__ int chunk_of(int sub, int cc)
{
    return (W == 512) ? cc * Cfg<W>::R + sub : sub * Cfg<W>::CPT + cc;
}

struct FusedLayer {
    const uint8_t *qw_umma;
    const uint32_t *qw_k4m;
    const float *cA, *cA_lo, *cB;
    const uint32_t *fxP, *fxQ, *fxB;
    const float *act;
    const int32_t *l1U, *l1V; // two-sided transform, layer 1: H_M applied to the two distinct weight-code sums
    int epi_mode;
    int c_off; // word offset of this layer's constants in the shared-memory constant area
};

struct FusedParams {
    const float *coords;
    float *out;
    long long n, n_tiles;
    int L, W, d_L, per_token;
    float qmaxf;
    int n_stages, resident;
    int bulk_xy;         // coords 16-byte aligned: whole tiles may arrive by bulk copy (width 512)
    int bulk_out;        // out 16-byte aligned: whole tiles may leave by bulk store (host-buffer variant)
    int const_words;
    int *status;
    unsigned long long wait_limit_ns; // every bounded wait gives up after this long (a handle setting)
    int skip_last_weights;            // test hook: the copy role leaves out the last layer's weights once
    FusedLayer layer[kMaxLayers];
    float gabor_c;                    // wavelet activation: s0 / omega0 (read by the GABOR instantiations only)
};

struct FusedParamsDump : FusedParams {
    DumpPtrs d;
};
template <bool DUMP> using ParamsOf = std::conditional_t<DUMP, FusedParamsDump, FusedParams>;

struct FusedState {
    FusedParams p;
    size_t smem_bytes;
    int sm_count;
};

// Shared-memory map (byte offsets from a 1024-byte aligned base).
struct SmemMap {
    uint32_t a_tile[2];
    uint32_t ring, last_w, consts, amax;
    uint32_t xy;         // [2 slots][4 threads of a row][128 rows] float2: coordinates fetched ahead
    uint32_t out_tile;   // [2 slots][128 rows][4] fp32: a tile's results before their bulk store (width <= 256)
    uint32_t acc_full;   // [2 slots][4 pieces]
    uint32_t acc_last;   // [2]
    uint32_t codes_full; // [2]
    uint32_t slot_sync;  // [2 slots][4 lane quadrants]
    uint32_t last_full, drain;
    uint32_t xy_full, xy_empty; // [2 slots] each: coordinates by bulk copy
    uint32_t out_sync;   // [2 slots]: the 128 threads that fill a slot's result buffer (host-buffer variant)
    uint32_t w_full, w_empty; // [kMaxStages] each
    uint32_t tmem_holder, abort_flag; // abort_flag: int flag + pad, then unsigned long long wait limit (ns)
    uint32_t total;
};

__host__ __device__ inline SmemMap smem_map(int W, int n_stages, int const_words)
{
    const int slots = (W == 512) ? 1 : 2;
    const uint32_t piece_bytes = (W == 512) ? 128u * 256u : (uint32_t)W * W;
    SmemMap m;
    uint32_t off = 0;
    m.a_tile[0] = off; off += kTile * W;
    m.a_tile[1] = off; if (slots == 2) off += kTile * W;
    m.ring = off; off += (uint32_t)n_stages * piece_bytes;
    m.last_w = off; off += 16 * W;
    m.consts = off; off += (uint32_t)const_words * 4;
    m.amax = off; off += 2 * 4 * kTile * 4;
    m.xy = off; off += (W != 512) ? 2 * 4 * kTile * 8 : kTile * 8; // per-thread entries, or one tile for the bulk copy
    m.out_tile = off; if (W != 512) off += 2 * kTile * 4 * 4; // placed here, among the 16-byte aligned areas: a bulk store reads it
    m.acc_full = off; off += 8 * 8;
    m.acc_last = off; off += 8 * 2;
    m.codes_full = off; off += 8 * 2;
    m.slot_sync = off; off += 8 * 8;
    m.last_full = off; off += 8;
    m.xy_full = off; if (W == 512) off += 16;
    m.xy_empty = off; if (W == 512) off += 16;
    m.out_sync = off; if (W != 512) off += 16;
    m.drain = off; off += 8;
    m.w_full = off; off += 8 * kMaxStages;
    m.w_empty = off; off += 8 * kMaxStages;
    m.tmem_holder = off; off += 8;
    m.abort_flag = off; off += 16; // flag word, then (8 bytes further) the wait limit in ns
    m.total = off;
    return m;
}

// Bounded wait.  Returns false when the wait ran out or another role already gave up.  Between
// tries the thread either sleeps (SLEEP_NS), so that a waiting warp leaves the issue slots to the
// working ones, or, with HINT_NS > 0, stays suspended inside the try itself for up to that long;
// the time limit and the abort flag are looked at every 64 tries.  Which form is faster was
// measured per role: the single-thread MMA and copy roles and the epilogue warps of the
// per-token kernels (two more barriers per layer) do better suspended, the epilogue warps of the
// per-tensor kernels sleeping.
constexpr int kHintNs = 2000;
// The launch's wait limit sits in shared memory next to the abort flag (written once in the
// kernel's prologue), so that it costs the waiting code no register.
__device__ __forceinline__ unsigned long long wait_limit_of(volatile int *abort_flag)
{
    return *reinterpret_cast<volatile unsigned long long *>(abort_flag + 2);
}
template <int SLEEP_NS, int HINT_NS = 0>
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = 0;
    for (uint32_t tries = 1;; ++tries) {
        if (HINT_NS > 0) {
            if (ptx::mbar_try_wait_hint(bar, parity, HINT_NS)) return true;
        } else {
            __nanosleep(SLEEP_NS);
            if (ptx::mbar_try_wait(bar, parity)) return true;
        }
        if ((tries & 63) == 0) {
            if (*abort_flag) return false;
            const unsigned long long now = ptx::globaltimer();
            if (t0 == 0) t0 = now;
            if (now - t0 > wait_limit_of(abort_flag)) {
                *abort_flag = 1;
                atomicExch(status, 1);
                return false;
            }
        }
    }
}
// The same for a whole warp: every lane takes the same decision.
template <bool SUSPEND>
__device__ __forceinline__ bool wait_bar_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status)
{
    return __all_sync(0xffffffffu, wait_bar<32, SUSPEND ? kHintNs : 0>(bar, parity, abort_flag, status));
}

// Two fp32 values in one 64-bit register pair, and the packed sm_100 arithmetic on them: one
// instruction, two IEEE round-to-nearest results (the same bits as two scalar operations).
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi)
{
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ f32x2 pack2u(uint32_t lo, uint32_t hi)
{
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ void unpack2u(f32x2 v, uint32_t &lo, uint32_t &hi) { asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(v)); }
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) { f32x2 r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) { f32x2 r; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) { f32x2 r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b)); return r; }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) { f32x2 r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c)); return r; }
// One butterfly on two independent pairs at once: (a, b) -> (a + b, a - b).
__device__ __forceinline__ void bfly2(f32x2 &a, f32x2 &b)
{
    const f32x2 x = a, y = b;
    a = add2(x, y);
    b = sub2(x, y);
}

// Round-half-even of two values to integer codes held in the low bytes: multiply by inv,
// (clamp,) add 1.5 * 2^23 - the sum rounds to the integer grid, ties to even, and its low
// mantissa bits are the two's complement code.  Same integers as
// __float2int_rn(clamp(v * inv, -qmax, qmax)).  With a per-token scale |v * inv| <= qmax
// (1 + 2^-23) already, so the clamp is skipped.  The clamp is sign(t) * min(|t|, qmax).
template <bool CLAMP> __device__ __forceinline__ void code_bits2(f32x2 v, f32x2 inv2, float qmaxf, uint32_t &b0, uint32_t &b1)
{
    f32x2 t = mul2(v, inv2);
    float lo, hi;
    unpack2(t, lo, hi);
    if (CLAMP) {
        asm("min.xorsign.abs.f32 %0, %0, %1;" : "+f"(lo) : "f"(qmaxf));
        asm("min.xorsign.abs.f32 %0, %0, %1;" : "+f"(hi) : "f"(qmaxf));
        unpack2u(add2(pack2(lo, hi), pack2(12582912.0f, 12582912.0f)), b0, b1);
    } else {
        // Scalar adds here: a packed multiply directly followed by a packed add was observed to be
        // merged into one fused multiply-add by the assembler, which rounds v * inv only once and
        // turns exact ties (x.5) the wrong way.  The product must be rounded to fp32 first.
        b0 = __float_as_uint(__fadd_rn(lo, 12582912.0f));
        b1 = __float_as_uint(__fadd_rn(hi, 12582912.0f));
    }
}
template <bool CLAMP> __device__ __forceinline__ uint32_t code_bits(float v, float inv, float qmaxf)
{
    float t = __fmul_rn(v, inv);
    if (CLAMP) asm("min.xorsign.abs.f32 %0, %0, %1;" : "+f"(t) : "f"(qmaxf));
    return __float_as_uint(__fadd_rn(t, 12582912.0f));
}
__device__ __forceinline__ uint32_t pack4(uint32_t b0, uint32_t b1, uint32_t b2, uint32_t b3)
{
    uint32_t lo = __byte_perm(b0, b1, 0x0040);
    uint32_t hi = __byte_perm(b2, b3, 0x0040);
    return __byte_perm(lo, hi, 0x5410);
}
// Store N (4, 8 or 16) consecutive-k codes of this thread's token, k0 a multiple of N, into the A
// operand tile: byte offset (k/16) * 2048 + row * 16 + k % 16.  w holds N/4 packed words.
template <int N> __device__ __forceinline__ void store_code_words(uint32_t a_tile, int row, int k0, const uint32_t *w)
{
    const uint32_t addr = a_tile + (k0 >> 4) * 2048 + row * 16 + (k0 & 15);
    if constexpr (N == 16)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
    else if constexpr (N == 8)
        asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(addr), "r"(w[0]), "r"(w[1]) : "memory");
    else
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(addr), "r"(w[0]) : "memory");
}
// Quantize G consecutive tensor-memory columns of chunk `ch` starting at column position p0 (even
// positions hold features p0/2 + k, odd positions features CH/2 + p0/2 + k) and store the codes.
template <int G, int CH, bool CLAMP, bool DUMP = false>
__device__ __forceinline__ void quantize_store(uint32_t a_tile, int row, int ch, int p0, const uint32_t *u, float inv, float qmaxf,
                                               int8_t *dump_row = nullptr)
{
    const f32x2 inv2 = pack2(inv, inv);
    uint32_t even[G / 2], odd[G / 2];
#pragma unroll
    for (int k = 0; k < G / 2; ++k) code_bits2<CLAMP>(pack2u(u[2 * k], u[2 * k + 1]), inv2, qmaxf, even[k], odd[k]);
    uint32_t we[G / 8], wo[G / 8];
#pragma unroll
    for (int j = 0; j < G / 8; ++j) {
        we[j] = pack4(even[4 * j], even[4 * j + 1], even[4 * j + 2], even[4 * j + 3]);
        wo[j] = pack4(odd[4 * j], odd[4 * j + 1], odd[4 * j + 2], odd[4 * j + 3]);
    }
    store_code_words<G / 2>(a_tile, row, ch * CH + p0 / 2, we);
    store_code_words<G / 2>(a_tile, row, ch * CH + CH / 2 + p0 / 2, wo);
    if constexpr (DUMP) {
        // the very words that went into the A operand tile, at their feature positions k
        if (dump_row) {
#pragma unroll
            for (int j = 0; j < G / 8; ++j) {
                *reinterpret_cast<uint32_t *>(dump_row + ch * CH + p0 / 2 + 4 * j) = we[j];
                *reinterpret_cast<uint32_t *>(dump_row + ch * CH + CH / 2 + p0 / 2 + 4 * j) = wo[j];
            }
        }
    }
}

template <int N> __device__ __forceinline__ void tmem_ld(uint32_t taddr, uint32_t (&v)[N])
{
    if constexpr (N == 8) ptx::tmem_ld8(taddr, v);
    else if constexpr (N == 16) ptx::tmem_ld16(taddr, v);
    else if constexpr (N == 32) ptx::tmem_ld32(taddr, v);
    else ptx::tmem_ld64(taddr, v);
}
template <int N> __device__ __forceinline__ void tmem_st(uint32_t taddr, const uint32_t (&v)[N])
{
    if constexpr (N == 8) ptx::tmem_st8(taddr, v);
    else if constexpr (N == 16) ptx::tmem_st16(taddr, v);
    else if constexpr (N == 32) ptx::tmem_st32(taddr, v);
    else ptx::tmem_st64(taddr, v);
}

__device__ __forceinline__ float4 lds128(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

// Pass 1 of one chunk, in place: v holds CH int32 accumulators (or nothing, for layer 1) on entry
// and, on exit, the fp32 activations after the butterfly stages with strides 1 .. CH/2.
// Tensor-memory column 2i of the chunk is feature i, column 2i+1 feature i + CH/2, so the
// register pair (v[2i], v[2i+1]) goes through the stages with strides 1 .. CH/4 as one packed
// value; the stride-CH/2 stage is the butterfly between its two halves.
// `sine8(j, out)` produces the four pairs 4j .. 4j+3.  The work is ordered as a software pipeline -
// the sines of group j+1 are issued before the stride-1/2 butterflies of group j, the stride-4/8
// butterflies follow every fourth group - so that the special-function unit (one sine per 8 issue
// cycles and scheduler) is fed evenly instead of in one burst per chunk.  Each element still goes
// through the stages in the order 1, 2, 4, ...: the sums are unchanged.
template <int CH, bool ROT, class Sine8> __device__ __forceinline__ void chunk_pipeline(uint32_t (&v)[CH], Sine8 sine8)
{
    constexpr int NP = CH / 2;
    f32x2 P[NP];
    if constexpr (!ROT) { // no rotation (plain uniform quantization): activations only
#pragma unroll
        for (int j = 0; j < NP / 4; ++j) sine8(j, &P[4 * j]);
#pragma unroll
        for (int i = 0; i < NP; ++i) unpack2u(P[i], v[2 * i], v[2 * i + 1]);
        return;
    }
    sine8(0, &P[0]);
#pragma unroll
    for (int j = 0; j < NP / 4; ++j) {
        if (j + 1 < NP / 4) sine8(j + 1, &P[4 * (j + 1)]);
        bfly2(P[4 * j], P[4 * j + 1]);
        bfly2(P[4 * j + 2], P[4 * j + 3]);
        bfly2(P[4 * j], P[4 * j + 2]);
        bfly2(P[4 * j + 1], P[4 * j + 3]);
        if ((j & 3) == 3) {
            const int base = 4 * (j - 3);
#pragma unroll
            for (int h = 4; h <= 8; h <<= 1) {
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    if ((i & h) == 0) bfly2(P[base + i], P[base + i + h]);
            }
        }
    }
#pragma unroll
    for (int h = 16; h < NP; h <<= 1) {
#pragma unroll
        for (int i = 0; i < NP; ++i)
            if ((i & h) == 0) bfly2(P[i], P[i + h]);
    }
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        float a, b;
        unpack2(P[i], a, b);
        v[2 * i] = __float_as_uint(__fadd_rn(a, b));
        v[2 * i + 1] = __float_as_uint(__fsub_rn(a, b));
    }
}

// Observing instantiation: four activations of tensor-memory columns col .. col+3 to the row of a
// [n][W] dump, each at its feature index.
template <int W> __device__ __forceinline__ void dump_y4(float *yrow, int col, f32x2 p0, f32x2 p1)
{
    if (!yrow) return;
    float y[4];
    unpack2(p0, y[0], y[1]);
    unpack2(p1, y[2], y[3]);
#pragma unroll
    for (int e = 0; e < 4; ++e) yrow[fused_feature(col + e, W)] = y[e];
}

// Hidden layer: dequantize + bias + sine of the CH columns starting at column m0.  Constants come
// from shared memory in column order: area A = cA, B = cB, C = cA_lo, each W words.
// TRACK (with EPI_SINE_FAST): *xmax receives the largest |phase| the thread met, for the caller's decision
// whether the chunk has to be redone under EPI_SINE_MIXED.  LIMIT: the limit of EPI_SINE_MIXED.
template <int W, int CH, bool PER_TOKEN, bool ROT, int MODE, bool DUMP = false, bool GABOR = false, bool TRACK = false>
__device__ __forceinline__ void hidden_chunk(uint32_t cbase, int m0, float s_x, uint32_t (&v)[CH], float *dump_y = nullptr,
                                             float gabor_c = 0.f, [[maybe_unused]] float *xmax = nullptr, [[maybe_unused]] float limit = 0.f)
{
    [[maybe_unused]] float xm = 0.f;
    chunk_pipeline<CH, ROT>(v, [&](int j, f32x2 *out) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int i = 8 * j + 4 * q; // four columns = two pairs
            const float4 a = lds128(cbase + (m0 + i) * 4);
            const float4 b = lds128(cbase + (W + m0 + i) * 4);
            if (MODE == EPI_SINE_FAST && !PER_TOKEN) {
                // x = fma(acc, cA, cB) for two columns at once, then the sine of each
                float x0, x1, x2, x3;
                unpack2(fma2(pack2((float)(int)v[i], (float)(int)v[i + 1]), pack2(a.x, a.y), pack2(b.x, b.y)), x0, x1);
                unpack2(fma2(pack2((float)(int)v[i + 2], (float)(int)v[i + 3]), pack2(a.z, a.w), pack2(b.z, b.w)), x2, x3);
                if constexpr (TRACK) xm = fmaxf(xm, fmaxf(fmaxf(fabsf(x0), fabsf(x1)), fmaxf(fabsf(x2), fabsf(x3))));
                out[2 * q] = pack2(sin_approx(x0), sin_approx(x1));
                out[2 * q + 1] = pack2(sin_approx(x2), sin_approx(x3));
            } else {
                float4 lo = make_float4(0.f, 0.f, 0.f, 0.f);
                if (MODE == EPI_SINE_WIDE || MODE == EPI_SINE_MIXED) lo = lds128(cbase + (2 * W + m0 + i) * 4);
                const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w}, lv[4] = {lo.x, lo.y, lo.z, lo.w};
                float y[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float c_hi = av[e], c_lo = lv[e];
                    if (PER_TOKEN) token_const(av[e], lv[e], s_x, c_hi, c_lo);
                    if constexpr (TRACK) { // EPI_SINE_FAST, keeping the phase
                        const float x = __fmaf_rn((float)(int)v[i + e], c_hi, bv[e]);
                        xm = fmaxf(xm, fabsf(x));
                        y[e] = sin_approx(x);
                    } else if constexpr (MODE == EPI_SINE_MIXED) {
                        y[e] = epilogue_mixed((float)(int)v[i + e], c_hi, c_lo, bv[e], limit);
                    } else {
                        y[e] = GABOR ? gabor_epilogue((float)(int)v[i + e], c_hi, c_lo, bv[e], gabor_c)
                                     : epilogue(MODE, (float)(int)v[i + e], c_hi, c_lo, bv[e]);
                    }
                }
                out[2 * q] = pack2(y[0], y[1]);
                out[2 * q + 1] = pack2(y[2], y[3]);
            }
            if constexpr (DUMP) dump_y4<W>(dump_y, m0 + i, out[2 * q], out[2 * q + 1]);
        }
    });
    if constexpr (TRACK) *xmax = xm;
}

// Layer 1 for the CH columns starting at column m0.  Fixed-point mode: areas A = P, B = B, C = Q.
// Float mode (per-token scales): A = cA, B = cB, C = cA_lo, D = the weight codes, one word per
// column, and acc = dp4a(codes of the token, codes of the column's feature).
template <int W, int CH, bool PER_TOKEN, bool ROT, bool DUMP = false, bool BOTH = false, bool GABOR = false>
__device__ __forceinline__ void layer1_chunk(uint32_t cbase, int m0, int qs, int qd, uint32_t qx, float s_x, uint32_t (&v)[CH],
                                             float *dump_y = nullptr, float gabor_c = 0.f)
{
    chunk_pipeline<CH, ROT>(v, [&](int j, f32x2 *out) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int i = 8 * j + 4 * q;
            const float4 A = lds128(cbase + (m0 + i) * 4);
            const float4 B = lds128(cbase + (W + m0 + i) * 4);
            const float4 Cc = lds128(cbase + (2 * W + m0 + i) * 4);
            const float Av[4] = {A.x, A.y, A.z, A.w}, Bv[4] = {B.x, B.y, B.z, B.w}, Cv[4] = {Cc.x, Cc.y, Cc.z, Cc.w};
            float y[4];
            if constexpr (!PER_TOKEN && !GABOR) {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    y[e] = sine_fixed(qs, qd, __float_as_uint(Av[e]), __float_as_uint(Cv[e]), __float_as_uint(Bv[e]));
            } else {
                const float4 wq = lds128(cbase + (3 * W + m0 + i) * 4);
                const float wv[4] = {wq.x, wq.y, wq.z, wq.w};
                float4 wq2 = make_float4(0.f, 0.f, 0.f, 0.f);
                if constexpr (BOTH) wq2 = lds128(cbase + (4 * W + m0 + i) * 4);
                const float wv2[4] = {wq2.x, wq2.y, wq2.z, wq2.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float c_hi = Av[e], c_lo = Cv[e]; // per-tensor scale (wavelet route): the constants hold s_x already
                    if (PER_TOKEN) token_const(Av[e], Cv[e], s_x, c_hi, c_lo);
                    // two-sided transform: areas D, E hold U' = H_M u and V' = H_M v (u, v: the sums of the weight
                    // codes that meet the two distinct input codes), so acc' = qs U' + qd V' needs no butterfly
                    const int acc = BOTH ? qs * (int)__float_as_uint(wv[e]) + qd * (int)__float_as_uint(wv2[e])
                                         : __dp4a((int)qx, (int)__float_as_uint(wv[e]), 0);
                    // (the wavelet's envelope needs the unwrapped phase, which the fixed-point route does not have)
                    y[e] = GABOR ? gabor_epilogue((float)acc, c_hi, c_lo, Bv[e], gabor_c) : epilogue(EPI_SINE_WIDE, (float)acc, c_hi, c_lo, Bv[e]);
                }
            }
            out[2 * q] = pack2(y[0], y[1]);
            out[2 * q + 1] = pack2(y[2], y[3]);
            if constexpr (DUMP) dump_y4<W>(dump_y, m0 + i, out[2 * q], out[2 * q + 1]);
        }
    });
}

// Everything a slot's threads need to finish a layer once their chunks are back in tensor memory.
struct SlotCtx {
    uint32_t taddr;      // TMEM address of this thread's lane, column 0 of the slot
    uint32_t a_tile;     // shared-memory address of the slot's A operand tile
    uint32_t bar_sync;   // mbarrier of the R warps that share this thread's 32 rows
    uint32_t bar_codes;  // "codes ready" mbarrier
    uint32_t amax_addr;  // shared memory: [R][128] floats for this slot
    uint32_t sync_parity;
    int row, sub;
    float qmaxf;
    volatile int *abort_flag;
    int *status;
};

template <bool SUSPEND> __device__ __forceinline__ bool slot_barrier(SlotCtx &c)
{
    ptx::mbar_arrive(c.bar_sync);
    bool ok = wait_bar_warp<SUSPEND>(c.bar_sync, c.sync_parity, c.abort_flag, c.status);
    c.sync_parity ^= 1;
    return ok;
}

// Passes 2 and 3: remaining butterfly stages across chunks, quantizer, store of the codes, and the
// arrival on the "codes ready" barrier.  Returns false if a wait ran out.  s_out receives the
// token's activation scale of the next layer.
template <int W, bool PER_TOKEN, bool ROT, bool DUMP = false>
__device__ __forceinline__ bool finish_layer(SlotCtx &c, float static_s, float static_inv, float &s_out, int8_t *dump_codes = nullptr)
{
    using C = Cfg<W>;
    constexpr int NCH = C::NCH, G = C::G, CH = C::CH;
    ptx::tmem_wait_st();
    ptx::tc_fence_before();
    if (!slot_barrier<PER_TOKEN>(c)) return false;
    ptx::tc_fence_after();
    float amax = 0.f;
#pragma unroll 1
    for (int gg = 0; gg < C::GPT; ++gg) {
        const int g = c.sub * C::GPT + gg;
        uint32_t u[NCH][G];
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) tmem_ld<G>(c.taddr + ch * CH + g * G, u[ch]);
        ptx::tmem_wait_ld();
        // strides CH, 2 CH, ...: the chunk index is the butterfly index; two columns per instruction
#pragma unroll
        for (int h = 1; h < (ROT ? NCH : 1); h <<= 1) {
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
                if ((ch & h) == 0) {
#pragma unroll
                    for (int i = 0; i < G; i += 2) {
                        f32x2 a = pack2u(u[ch][i], u[ch][i + 1]), b = pack2u(u[ch + h][i], u[ch + h][i + 1]);
                        bfly2(a, b);
                        unpack2u(a, u[ch][i], u[ch][i + 1]);
                        unpack2u(b, u[ch + h][i], u[ch + h][i + 1]);
                    }
                }
            }
        }
        if (PER_TOKEN) {
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
#pragma unroll
                for (int i = 0; i < G; ++i) amax = fmaxf(amax, fabsf(__uint_as_float(u[ch][i])));
                tmem_st<G>(c.taddr + ch * CH + g * G, u[ch]);
            }
        } else {
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) quantize_store<G, CH, true, DUMP>(c.a_tile, c.row, ch, g * G, u[ch], static_inv, c.qmaxf, dump_codes);
        }
    }
    if (!PER_TOKEN) {
        s_out = static_s;
    } else {
        // combine the row's absmax over the R threads that share it
        asm volatile("st.shared.f32 [%0], %1;" ::"r"(c.amax_addr + (c.sub * kTile + c.row) * 4), "f"(amax) : "memory");
        ptx::tmem_wait_st();
        ptx::tc_fence_before();
        if (!slot_barrier<PER_TOKEN>(c)) return false;
        ptx::tc_fence_after();
#pragma unroll
        for (int r = 0; r < C::R; ++r) {
            float o;
            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(o) : "r"(c.amax_addr + (r * kTile + c.row) * 4));
            amax = fmaxf(amax, o);
        }
        float s, inv;
        scales_of(amax, c.qmaxf, s, inv);
        s_out = s;
#pragma unroll 1
        for (int gg = 0; gg < C::GPT; ++gg) {
            const int g = c.sub * C::GPT + gg;
            uint32_t u[NCH][G];
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) tmem_ld<G>(c.taddr + ch * CH + g * G, u[ch]);
            ptx::tmem_wait_ld();
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) quantize_store<G, CH, false, DUMP>(c.a_tile, c.row, ch, g * G, u[ch], inv, c.qmaxf, dump_codes);
        }
    }
    ptx::fence_proxy_async();
    ptx::tc_fence_before();
    ptx::mbar_arrive(c.bar_codes);
    return true;
}

// Calibration instantiation (per-tensor activation scales, Section III-C's run-time statistic taken
// once): in place of the quantizer, the maximum of |x~| over the tile's valid tokens goes to the
// calibrated layer's act[0] (atomic maximum on the bit pattern: non-negative floats order as
// integers).  Same barrier, loads and butterfly stages as finish_layer up to that point.
template <int W, bool ROT> __device__ __forceinline__ bool calib_finish(SlotCtx &c, bool valid, float *act)
{
    using C = Cfg<W>;
    constexpr int NCH = C::NCH, G = C::G, CH = C::CH;
    ptx::tmem_wait_st();
    ptx::tc_fence_before();
    if (!slot_barrier<false>(c)) return false;
    ptx::tc_fence_after();
    float amax = 0.f;
#pragma unroll 1
    for (int gg = 0; gg < C::GPT; ++gg) {
        const int g = c.sub * C::GPT + gg;
        uint32_t u[NCH][G];
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) tmem_ld<G>(c.taddr + ch * CH + g * G, u[ch]);
        ptx::tmem_wait_ld();
#pragma unroll
        for (int h = 1; h < (ROT ? NCH : 1); h <<= 1) {
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
                if ((ch & h) == 0) {
#pragma unroll
                    for (int i = 0; i < G; i += 2) {
                        f32x2 a = pack2u(u[ch][i], u[ch][i + 1]), b = pack2u(u[ch + h][i], u[ch + h][i + 1]);
                        bfly2(a, b);
                        unpack2u(a, u[ch][i], u[ch][i + 1]);
                        unpack2u(b, u[ch + h][i], u[ch + h][i + 1]);
                    }
                }
            }
        }
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
#pragma unroll
            for (int i = 0; i < G; ++i) amax = fmaxf(amax, fabsf(__uint_as_float(u[ch][i])));
        }
    }
    if (!valid) amax = 0.f; // rows past the end of the coordinate set do not count
#pragma unroll
    for (int o = 16; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((c.row & 31) == 0) atomicMax(reinterpret_cast<unsigned int *>(act), __float_as_uint(amax));
    // the next tile's first layer writes these tensor-memory columns: every warp of the row group
    // must have finished reading them
    ptx::tc_fence_before();
    if (!slot_barrier<false>(c)) return false;
    ptx::tc_fence_after();
    return true;
}

// Observing instantiation: the int32 accumulators of CH tensor-memory columns starting at column
// m0, as they were read from tensor memory, to the row of an [n][W] dump at their feature indices.
template <int W, int CH> __device__ __forceinline__ void dump_acc_chunk(int32_t *arow, int m0, const uint32_t (&v)[CH])
{
    if (!arow) return;
#pragma unroll
    for (int i = 0; i < CH; ++i) arow[fused_feature(m0 + i, W)] = (int32_t)v[i];
}

// Two-sided transform (Eq. 4-5 literally): the layer output is z = H_M (s_w s_x acc) + b.  With one
// weight scale per tensor the rotation acts on the integers, acc' = H_M acc, exactly (32-bit
// wrap-around arithmetic; the host has checked that no value can leave the int32 range).  First the
// stages inside a chunk: tensor-memory column 2i is feature i, column 2i+1 feature i + CH/2.
template <int CH> __device__ __forceinline__ void int_butterfly_chunk(uint32_t (&v)[CH])
{
    constexpr int NP = CH / 2;
#pragma unroll
    for (int h = 1; h < NP; h <<= 1) {
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            if ((i & h) == 0) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const uint32_t a = v[2 * i + e], b = v[2 * (i + h) + e];
                    v[2 * i + e] = a + b;
                    v[2 * (i + h) + e] = a - b;
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        const uint32_t a = v[2 * i], b = v[2 * i + 1];
        v[2 * i] = a + b;
        v[2 * i + 1] = a - b;
    }
}
// ... then the stages across chunks, on groups of G positions of every chunk (as pass 2 does for
// the forward rotation), in place in tensor memory.  Both sides of it are barriers of the R warps
// that share the rows.  Returns false if a wait ran out.
template <int W> __device__ __forceinline__ bool int_butterfly_across(SlotCtx &c)
{
    using C = Cfg<W>;
    constexpr int NCH = C::NCH, G = C::G, CH = C::CH;
    ptx::tmem_wait_st();
    ptx::tc_fence_before();
    if (!slot_barrier<false>(c)) return false;
    ptx::tc_fence_after();
#pragma unroll 1
    for (int gg = 0; gg < C::GPT; ++gg) {
        const int g = c.sub * C::GPT + gg;
        uint32_t u[NCH][G];
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) tmem_ld<G>(c.taddr + ch * CH + g * G, u[ch]);
        ptx::tmem_wait_ld();
#pragma unroll
        for (int h = 1; h < NCH; h <<= 1) {
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
                if ((ch & h) == 0) {
#pragma unroll
                    for (int i = 0; i < G; ++i) {
                        const uint32_t a = u[ch][i], b = u[ch + h][i];
                        u[ch][i] = a + b;
                        u[ch + h][i] = a - b;
                    }
                }
            }
        }
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) tmem_st<G>(c.taddr + ch * CH + g * G, u[ch]);
    }
    ptx::tmem_wait_st();
    ptx::tc_fence_before();
    if (!slot_barrier<false>(c)) return false;
    ptx::tc_fence_after();
    return true;
}

template <int W, bool PER_TOKEN, bool ROT, bool SPREAD, bool AHEAD, bool DUMP, bool BOTH, bool CALIB, bool GABOR, bool MIXED>
__device__ void epilogue_role(const ParamsOf<DUMP> &p, const SmemMap &sm, uint32_t smem_base, int warp, int lane,
                              uint32_t tmem_base, volatile int *abort_flag)
{
    using C = Cfg<W>;
    constexpr int CH = C::CH;
    const int slot = warp / (4 * C::R);
    const int quad = warp & 3;
    const int sub = (warp % (4 * C::R)) >> 2;
    SlotCtx c;
    c.row = quad * 32 + lane;
    c.sub = sub;
    c.taddr = tmem_base + (uint32_t)(slot * C::TMEM_COLS_PER_SLOT) + ((uint32_t)(quad * 32) << 16);
    c.a_tile = smem_base + sm.a_tile[slot];
    c.bar_sync = smem_base + sm.slot_sync + 8 * (slot * 4 + quad);
    c.bar_codes = smem_base + sm.codes_full + 8 * slot;
    c.amax_addr = smem_base + sm.amax + slot * (4 * kTile * 4);
    c.sync_parity = 0;
    c.qmaxf = p.qmaxf;
    c.abort_flag = abort_flag;
    c.status = p.status;
    const uint32_t bar_acc = smem_base + sm.acc_full + 8 * (slot * 4);
    const uint32_t bar_last = smem_base + sm.acc_last + 8 * slot;
    const uint32_t consts = smem_base + sm.consts;
    const uint32_t xy_addr = smem_base + sm.xy + (uint32_t)(((slot * 4 + sub) * kTile + c.row) * 8);
    uint32_t acc_parity = 0, last_parity = 0;
    [[maybe_unused]] uint32_t xy_k = 0; // tiles taken from the bulk-copy buffer so far
    [[maybe_unused]] uint32_t out_parity = 0;
    const FusedLayer &l1 = p.layer[0];
    const float qmaxf = p.qmaxf;

    if (C::SLOTS == 2 && slot == 1 && tile_index<SPREAD>(0, 1, 2) < p.n_tiles && p.resident) {
        // Start the second slot about half a layer period after the first, so that one slot's
        // sine-heavy pass 1 and MMA wait fall on the other slot's pass 2 instead of both slots
        // asking for the same pipe at the same time.  The offset then keeps itself.  Not when the
        // weights are streamed: there both slots should consume a slab while it is in the ring.
        const unsigned long long t0 = ptx::globaltimer(), delay = (3500ull * W * W) / (256 * 256);
        while (ptx::globaltimer() - t0 < delay) __nanosleep(64);
    }
    for (long long r = 0;; ++r) {
        const long long tile = tile_index<SPREAD>(r, slot, C::SLOTS);
        if (tile >= p.n_tiles) break;
        const long long tok = tile * kTile + c.row;
        const bool valid = tok < p.n;

        // ---------------- layer 1 on the CUDA cores: x~ = H_4 [x, y, 0, 0]
        float x = 0.f, y = 0.f;
        if constexpr (C::BULK_XY) {
            if (p.bulk_xy && (tile + 1) * kTile <= p.n) {
                // the whole tile was brought to shared memory by one bulk copy, a tile ahead
                if (!wait_bar_warp<PER_TOKEN>(smem_base + sm.xy_full + 8 * slot, xy_k & 1u, abort_flag, p.status)) return;
                ++xy_k;
                asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(x), "=f"(y) : "r"(smem_base + sm.xy + (uint32_t)((slot * kTile + c.row) * 8)));
                // The arrival below hands the buffer back to the copy warp, whose next bulk copy (async
                // proxy) overwrites it.  The arrival does not wait for this thread's load to have been
                // performed: with the load/store unit backed up (the observing instantiation's stores) the
                // load was seen to return the NEXT tile's coordinates.  The proxy fence orders the read
                // before everything after it.
                ptx::fence_proxy_async();
                ptx::mbar_arrive(smem_base + sm.xy_empty + 8 * slot);
            } else if (valid) { // ragged last tile, or coordinates not 16-byte aligned
                float2 xy = __ldg(reinterpret_cast<const float2 *>(p.coords) + tok);
                x = xy.x; y = xy.y;
            }
        } else
        if (!AHEAD || r == 0) {
            if (valid) {
                float2 xy = __ldg(reinterpret_cast<const float2 *>(p.coords) + tok);
                x = xy.x; y = xy.y;
            }
        } else {
            // copied into shared memory by this thread while the previous tile was in its hidden layers
            asm volatile("cp.async.wait_all;" ::: "memory");
            if (valid) asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(x), "=f"(y) : "r"(xy_addr));
        }
        float e0 = x, e1 = y, e2 = 0.f, e3 = 0.f;
        if (ROT) {
            float r0 = __fadd_rn(x, y), r1 = __fsub_rn(x, y), r2 = __fadd_rn(0.f, 0.f), r3 = __fsub_rn(0.f, 0.f);
            e0 = __fadd_rn(r0, r2); e2 = __fsub_rn(r0, r2); e1 = __fadd_rn(r1, r3); e3 = __fsub_rn(r1, r3);
        }
        float s_x, inv_x;
        if (PER_TOKEN) {
            float a = fmaxf(fmaxf(fabsf(e0), fabsf(e1)), fmaxf(fabsf(e2), fabsf(e3)));
            scales_of(a, qmaxf, s_x, inv_x);
        } else {
            s_x = __ldg(l1.act + 1);
            inv_x = __ldg(l1.act + 2);
        }
        const uint32_t b0 = code_bits<true>(e0, inv_x, qmaxf), b1 = code_bits<true>(e1, inv_x, qmaxf);
        const uint32_t qx = pack4(b0, b1, code_bits<true>(e2, inv_x, qmaxf), code_bits<true>(e3, inv_x, qmaxf));
        const int qs = (int)b0 - 0x4B400000, qd = (int)b1 - 0x4B400000;
        float next_s = 1.f, next_inv = 0.f;
        if (!PER_TOKEN) {
            next_s = __ldg(p.layer[1].act + 1);
            next_inv = __ldg(p.layer[1].act + 2);
        }
        // Observing instantiation: where this thread's token writes its per-layer values (null: skip)
        [[maybe_unused]] float *dY = nullptr;
        [[maybe_unused]] int8_t *dC = nullptr;
        if constexpr (DUMP) {
            if (valid) {
                if (sub == 0) {
                    if (p.d.X[0]) reinterpret_cast<float4 *>(p.d.X[0])[tok] = make_float4(x, y, 0.f, 0.f);
                    if (p.d.codes[0]) reinterpret_cast<uint32_t *>(p.d.codes[0])[tok] = qx;
                    if (p.d.s_x[0]) p.d.s_x[0][tok] = s_x;
                }
                dY = p.d.Y[0] ? p.d.Y[0] + tok * W : nullptr;
                dC = p.d.codes[1] ? p.d.codes[1] + tok * W : nullptr;
            }
        }
#pragma unroll
        for (int cc = 0; cc < C::CPT; ++cc) {
            const int ch = chunk_of<W>(sub, cc);
            uint32_t v[CH];
            if constexpr (DUMP) {
                // the first layer's accumulators are never formed on the fixed-point route (the phase is
                // built from the two distinct codes directly); the dump states them: codes . weight codes
                if (valid && p.d.acc[0]) {
                    for (int i = 0; i < CH; ++i) {
                        const int m = fused_feature(ch * CH + i, W);
                        p.d.acc[0][tok * W + m] = __dp4a((int)qx, (int)__ldg(l1.qw_k4m + m), 0);
                    }
                }
            }
            layer1_chunk<W, CH, PER_TOKEN, ROT, DUMP, BOTH, GABOR>(consts + l1.c_off * 4, ch * CH, qs, qd, qx, s_x, v, dY, p.gabor_c);
            tmem_st<CH>(c.taddr + ch * CH, v);
        }
        if constexpr (CALIB) {
            // calibration of layer p.L: the network is run up to that layer's rotated input
            if (p.L == 2) {
                if (!calib_finish<W, ROT>(c, valid, const_cast<float *>(p.layer[1].act))) return;
                continue;
            }
        }
        if (!finish_layer<W, PER_TOKEN, ROT, DUMP>(c, next_s, next_inv, s_x, dC)) return;
        if constexpr (DUMP) {
            if (valid && sub == 0 && p.d.s_x[1]) p.d.s_x[1][tok] = s_x;
        }
        if constexpr (AHEAD) {
            // The next tile's coordinates start their way into shared memory now.  An asynchronous
            // copy holds neither a register nor one of the warp's dependency barriers while it is in
            // flight (a plain load issued this early slowed the layers down: they wait on the barrier
            // it occupies).  Not earlier than this: at the start of a launch every tile's first fetch
            // is under way.  Only for coordinates in device memory: from mapped host memory the
            // 8-byte asynchronous copies were slower than the plain load at the tile's start.
            const long long tok_next = tile_index<SPREAD>(r + 1, slot, C::SLOTS) * kTile + c.row;
            if (tok_next < p.n)
                asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(xy_addr), "l"(reinterpret_cast<const float2 *>(p.coords) + tok_next) : "memory");
        }

        // ---------------- layers 2 .. L on the tensor core
        for (int l = 2; l < p.L; ++l) {
            const FusedLayer &ly = p.layer[l - 1];
            if (!wait_bar_warp<PER_TOKEN>(bar_acc, acc_parity, abort_flag, p.status)) return;
            if constexpr (C::NHALF == 1) acc_parity ^= 1;
            ptx::tc_fence_after();
            if (!PER_TOKEN) {
                next_s = __ldg(p.layer[l].act + 1);
                next_inv = __ldg(p.layer[l].act + 2);
            }
            const uint32_t cbase = consts + ly.c_off * 4;
            const bool fast = ly.epi_mode == EPI_SINE_FAST;
            if constexpr (BOTH) {
                // pass 0: acc' = H_W acc on the integers, in place in tensor memory
#pragma unroll
                for (int cc = 0; cc < C::CPT; ++cc) {
                    const int ch = chunk_of<W>(sub, cc);
                    if constexpr (C::NHALF == 2) {
                        if (cc == 1) {
                            if (!wait_bar_warp<PER_TOKEN>(bar_acc + 8, acc_parity, abort_flag, p.status)) return;
                            acc_parity ^= 1;
                            ptx::tc_fence_after();
                        }
                    }
                    uint32_t v[CH];
                    tmem_ld<CH>(c.taddr + ch * CH, v);
                    ptx::tmem_wait_ld();
                    if constexpr (DUMP) dump_acc_chunk<W, CH>((valid && p.d.acc[l - 1]) ? p.d.acc[l - 1] + tok * W : nullptr, ch * CH, v);
                    int_butterfly_chunk<CH>(v);
                    tmem_st<CH>(c.taddr + ch * CH, v);
                }
                if (!int_butterfly_across<W>(c)) return;
            }
#pragma unroll
            for (int cc = 0; cc < C::CPT; ++cc) {
                const int ch = chunk_of<W>(sub, cc);
                if constexpr (C::NHALF == 2 && !BOTH) {
                    // width 512: the thread's second chunk lies in the second half of the output columns,
                    // whose MMAs run while the first chunk is worked on
                    if (cc == 1) {
                        if (!wait_bar_warp<PER_TOKEN>(bar_acc + 8, acc_parity, abort_flag, p.status)) return;
                        acc_parity ^= 1;
                        ptx::tc_fence_after();
                    }
                }
                uint32_t v[CH];
                tmem_ld<CH>(c.taddr + ch * CH, v);
                ptx::tmem_wait_ld();
                if constexpr (DUMP) {
                    dY = (valid && p.d.Y[l - 1]) ? p.d.Y[l - 1] + tok * W : nullptr;
                    if constexpr (!BOTH) dump_acc_chunk<W, CH>((valid && p.d.acc[l - 1]) ? p.d.acc[l - 1] + tok * W : nullptr, ch * CH, v);
                }
                if (fast) {
                    hidden_chunk<W, CH, PER_TOKEN, ROT, EPI_SINE_FAST, DUMP>(cbase, ch * CH, s_x, v, dY);
                } else {
                    [[maybe_unused]] bool done = false;
                    if constexpr ((MIXED || BOTH) && !GABOR) {
                        if (ly.epi_mode == EPI_SINE_MIXED) {
                            // No bound says that the short route is accurate enough for this layer, but the phases
                            // that are actually met mostly are: take it, keep the largest |phase|, and redo the
                            // chunk value by value (accumulators are still in tensor memory) only if a warp met one
                            // beyond the limit.  The per-value rule gives the same bits either way.
                            constexpr float kLimit = BOTH ? kMixedPhaseLimitBoth : PER_TOKEN ? kFastPhaseLimitPerToken : kFastPhaseLimit;
                            float xm = 0.f;
                            hidden_chunk<W, CH, PER_TOKEN, ROT, EPI_SINE_FAST, DUMP, false, true>(cbase, ch * CH, s_x, v, dY, 0.f, &xm);
                            if (!__all_sync(0xffffffffu, xm <= kLimit)) {
                                tmem_ld<CH>(c.taddr + ch * CH, v);
                                ptx::tmem_wait_ld();
                                hidden_chunk<W, CH, PER_TOKEN, ROT, EPI_SINE_MIXED, DUMP>(cbase, ch * CH, s_x, v, dY, 0.f, nullptr, kLimit);
                            }
                            done = true;
                        }
                    }
                    if (!done) hidden_chunk<W, CH, PER_TOKEN, ROT, EPI_SINE_WIDE, DUMP, GABOR>(cbase, ch * CH, s_x, v, dY, p.gabor_c);
                }
                tmem_st<CH>(c.taddr + ch * CH, v);
            }
            if constexpr (DUMP) dC = (valid && p.d.codes[l]) ? p.d.codes[l] + tok * W : nullptr;
            if constexpr (CALIB) {
                if (l == p.L - 1) {
                    if (!calib_finish<W, ROT>(c, valid, const_cast<float *>(p.layer[l].act))) return;
                    continue;
                }
            }
            if (!finish_layer<W, PER_TOKEN, ROT, DUMP>(c, next_s, next_inv, s_x, dC)) return;
            if constexpr (DUMP) {
                if (valid && sub == 0 && p.d.s_x[l]) p.d.s_x[l][tok] = s_x;
            }
        }
        if constexpr (!CALIB) {
            const FusedLayer &ly = p.layer[p.L - 1];
            if (!wait_bar_warp<PER_TOKEN>(bar_last, last_parity, abort_flag, p.status)) return;
            last_parity ^= 1;
            ptx::tc_fence_after();
            if (sub == 0) {
                uint32_t u[4];
                ptx::tmem_ld4(c.taddr, u);
                ptx::tmem_wait_ld();
                [[maybe_unused]] uint32_t raw[4] = {u[0], u[1], u[2], u[3]};
                if constexpr (BOTH) { // z = H_4 (s_w s_x acc) + b over the four padded outputs, on the integers
                    const uint32_t a0 = u[0] + u[1], a1 = u[0] - u[1], a2 = u[2] + u[3], a3 = u[2] - u[3];
                    u[0] = a0 + a2; u[2] = a0 - a2; u[1] = a1 + a3; u[3] = a1 - a3;
                }
                // Host-buffer variant: a whole tile's results (128 x d_L floats, contiguous in `out`) are
                // collected in shared memory and leave by one bulk store: over the host link one large
                // write instead of 128 x d_L four-byte ones.  The slot's 128 sub-0 threads meet on an
                // mbarrier (bounded wait, like every other) before and after filling the buffer; its
                // first thread issues the store.
                const bool by_bulk = !AHEAD && !C::BULK_XY && p.bulk_out && (tile + 1) * kTile <= p.n;
                const uint32_t ot = smem_base + sm.out_tile + (uint32_t)(slot * kTile * 16);
                if (by_bulk) {
                    if (c.row == 0) ptx::bulk_wait_read(); // the previous tile's store has read the buffer
                    ptx::mbar_arrive(smem_base + sm.out_sync + 8 * slot);
                    if (!wait_bar_warp<PER_TOKEN>(smem_base + sm.out_sync + 8 * slot, out_parity, abort_flag, p.status)) return;
                    out_parity ^= 1;
                }
                if constexpr (DUMP) {
                    // all four padded outputs of the last layer: accumulators and z = c acc + b
                    if (valid) {
#pragma unroll
                        for (int m = 0; m < 4; ++m) {
                            float c_hi = __ldg(ly.cA + m);
                            if (PER_TOKEN) c_hi = __fmul_rn(c_hi, s_x);
                            if (p.d.acc[p.L - 1]) p.d.acc[p.L - 1][tok * 4 + m] = (int32_t)raw[m];
                            if (p.d.Y[p.L - 1]) p.d.Y[p.L - 1][tok * 4 + m] = epilogue(EPI_LINEAR, (float)(int)u[m], c_hi, 0.f, __ldg(ly.cB + m));
                        }
                    }
                }
                if (valid) {
#pragma unroll
                    for (int m = 0; m < 4; ++m) {
                        if (m < p.d_L) {
                            float c_hi = __ldg(ly.cA + m), c_lo = 0.f;
                            if (PER_TOKEN) c_hi = __fmul_rn(c_hi, s_x);
                            const float yv = epilogue(EPI_LINEAR, (float)(int)u[m], c_hi, c_lo, __ldg(ly.cB + m));
                            if (by_bulk) asm volatile("st.shared.f32 [%0], %1;" ::"r"(ot + (uint32_t)((c.row * p.d_L + m) * 4)), "f"(yv) : "memory");
                            else p.out[tok * p.d_L + m] = yv;
                        }
                    }
                }
                if (by_bulk) {
                    ptx::fence_proxy_async();
                    ptx::mbar_arrive(smem_base + sm.out_sync + 8 * slot);
                    if (!wait_bar_warp<PER_TOKEN>(smem_base + sm.out_sync + 8 * slot, out_parity, abort_flag, p.status)) return;
                    out_parity ^= 1;
                    if (c.row == 0) ptx::bulk_s2g(p.out + tile * kTile * p.d_L, ot, (uint32_t)(kTile * p.d_L * 4));
                }
            }
            ptx::tc_fence_before();
        }
    }
    if (!AHEAD && !C::BULK_XY && sub == 0 && c.row == 0) ptx::bulk_wait_all(); // the last tiles' stores
}

template <int W, bool SPREAD, bool CALIB>
__device__ void mma_role(const FusedParams &p, const SmemMap &sm, uint32_t smem_base, uint32_t tmem_base,
                         volatile int *abort_flag)
{
    using C = Cfg<W>;
    uint32_t codes_parity[2] = {0, 0};
    const uint32_t idesc_hidden = ptx::idesc_i8(kTile, C::NW), idesc_last = ptx::idesc_i8(kTile, 16);
    const uint32_t slab = C::PIECE_BYTES;
    // each K step of 32 advances a descriptor's start-address field (bits 0-13, 16-byte units) by
    // two core-matrix columns
    const uint64_t a_step = (uint64_t)((2 * kTile * 16) >> 4);
    long long use = 0; // ring uses so far (streaming mode)
    bool ok = true;
    for (long long r = 0; ok; ++r) {
        if (tile_index<SPREAD>(r, 0, C::SLOTS) >= p.n_tiles) break;
        const int active = (C::SLOTS == 2 && tile_index<SPREAD>(r, 1, C::SLOTS) < p.n_tiles) ? 2 : 1;
        for (int l = 2; l < p.L && ok; ++l) {
            if constexpr (C::NHALF == 2) {
                // width 512: eight pieces per layer, the four k-pieces of output columns 0..255 first;
                // each half of the accumulator is committed on its own barrier as soon as it is complete
                for (int pc = 0; pc < C::PIECES && ok; ++pc) {
                    const int half = pc / C::KSLABS, ksl = pc % C::KSLABS;
                    const int stage = (int)(use % p.n_stages);
                    const uint32_t par = (uint32_t)((use / p.n_stages) & 1);
                    if (!wait_bar<0, kHintNs>(smem_base + sm.w_full + 8 * stage, par, abort_flag, p.status)) { ok = false; break; }
                    if (pc == 0) {
                        if (!wait_bar<0, kHintNs>(smem_base + sm.codes_full, codes_parity[0], abort_flag, p.status)) { ok = false; break; }
                        codes_parity[0] ^= 1;
                        ptx::tc_fence_after();
                    }
                    const uint32_t b_addr = smem_base + sm.ring + (uint32_t)stage * C::PIECE_BYTES;
                    const uint64_t ad0 = ptx::smem_desc(smem_base + sm.a_tile[0] + ksl * (C::SLABK / 16) * (kTile * 16), kTile * 16, 128);
                    const uint32_t d = tmem_base + (uint32_t)(half * C::NW);
                    const uint64_t bd0 = ptx::smem_desc(b_addr, C::NW * 16, 128);
                    const uint64_t b_step = (uint64_t)((2 * C::NW * 16) >> 4);
#pragma unroll
                    for (int ks = 0; ks < C::SLABK / 32; ++ks)
                        ptx::mma_i8(d, ad0 + ks * a_step, bd0 + ks * b_step, idesc_hidden, (ksl > 0 || ks > 0) ? 1u : 0u);
                    if (ksl == C::KSLABS - 1) ptx::mma_commit(smem_base + sm.acc_full + 8 * half);
                    ptx::mma_commit(smem_base + sm.w_empty + 8 * stage);
                    ++use;
                }
                continue;
            }
            for (int ksl = 0; ksl < C::KSLABS && ok; ++ksl) {
                const int slab_id = (l - 2) * C::KSLABS + ksl;
                const int stage = p.resident ? slab_id : (int)(use % p.n_stages);
                const uint32_t par = p.resident ? 0u : (uint32_t)((use / p.n_stages) & 1);
                if (!wait_bar<0, kHintNs>(smem_base + sm.w_full + 8 * stage, par, abort_flag, p.status)) { ok = false; break; }
                const uint32_t b_addr = smem_base + sm.ring + (uint32_t)stage * slab;
                for (int s = 0; s < active; ++s) {
                    if (ksl == 0) {
                        if (!wait_bar<0, kHintNs>(smem_base + sm.codes_full + 8 * s, codes_parity[s], abort_flag, p.status)) { ok = false; break; }
                        codes_parity[s] ^= 1;
                        ptx::tc_fence_after();
                    }
                    const uint64_t ad0 = ptx::smem_desc(smem_base + sm.a_tile[s] + ksl * (C::SLABK / 16) * (kTile * 16), kTile * 16, 128);
#pragma unroll
                    for (int half = 0; half < C::NHALF; ++half) {
                        const uint32_t d = tmem_base + (uint32_t)(s * C::TMEM_COLS_PER_SLOT + half * C::NW);
                        const uint64_t bd0 = ptx::smem_desc(b_addr + half * C::NW * 16, W * 16, 128);
                        const uint64_t b_step = (uint64_t)((2 * W * 16) >> 4);
#pragma unroll
                        for (int ks = 0; ks < C::SLABK / 32; ++ks)
                            ptx::mma_i8(d, ad0 + ks * a_step, bd0 + ks * b_step, idesc_hidden, (ksl > 0 || ks > 0) ? 1u : 0u);
                    }
                    if (ksl == C::KSLABS - 1) ptx::mma_commit(smem_base + sm.acc_full + 8 * (s * 4));
                }
                if (!ok) break;
                if (!p.resident) {
                    ptx::mma_commit(smem_base + sm.w_empty + 8 * stage);
                    ++use;
                }
            }
        }
        if (!ok) break;
        if constexpr (CALIB) continue; // the calibrated layer itself is not computed
        // last layer: N = 16, its weights stay in shared memory
        if (!wait_bar<0, kHintNs>(smem_base + sm.last_full, 0, abort_flag, p.status)) { ok = false; break; }
        for (int s = 0; s < active; ++s) {
            if (!wait_bar<0, kHintNs>(smem_base + sm.codes_full + 8 * s, codes_parity[s], abort_flag, p.status)) { ok = false; break; }
            codes_parity[s] ^= 1;
            ptx::tc_fence_after();
            const uint32_t d = tmem_base + (uint32_t)(s * C::TMEM_COLS_PER_SLOT);
            const uint64_t ad0 = ptx::smem_desc(smem_base + sm.a_tile[s], kTile * 16, 128);
            const uint64_t bd0 = ptx::smem_desc(smem_base + sm.last_w, 16 * 16, 128);
            const uint64_t b_step = (uint64_t)((2 * 16 * 16) >> 4);
#pragma unroll
            for (int ks = 0; ks < W / 32; ++ks)
                ptx::mma_i8(d, ad0 + ks * a_step, bd0 + ks * b_step, idesc_last, ks > 0 ? 1u : 0u);
            ptx::mma_commit(smem_base + sm.acc_last + 8 * s);
        }
    }
    if (!ok) { // give the MMAs already issued a bounded time to finish before TMEM is released
        ptx::mma_commit(smem_base + sm.drain);
        const unsigned long long t0 = ptx::globaltimer();
        while (!ptx::mbar_try_wait(smem_base + sm.drain, 0) && ptx::globaltimer() - t0 < wait_limit_of(abort_flag)) {}
    }
}

template <int W, bool SPREAD, bool CALIB>
__device__ void load_role(const FusedParams &p, const SmemMap &sm, uint32_t smem_base, volatile int *abort_flag)
{
    using C = Cfg<W>;
    const uint32_t slab = C::PIECE_BYTES;
    // (test hook: with skip_last_weights set the copy is left out and nothing ever completes
    // last_full, so the waits for it run out, the abort path runs and the kernel returns)
    if (!p.skip_last_weights && !CALIB) {
        ptx::mbar_expect_tx(smem_base + sm.last_full, 16 * W);
        ptx::bulk_g2s(smem_base + sm.last_w, p.layer[p.L - 1].qw_umma, 16 * W, smem_base + sm.last_full);
    }
    const int slabs = (p.L - 2) * C::PIECES; // per tile round
    if (slabs <= 0) return;
    long long rounds = 0;
    for (long long r = 0;; ++r) {
        if (tile_index<SPREAD>(r, 0, C::SLOTS) >= p.n_tiles) break;
        ++rounds;
    }
    const long long total = p.resident ? slabs : rounds * slabs;
    long long issued = 0;
    bool ok = true;
    for (long long i = 0; i < total; ++i) {
        const int stage = (int)(i % p.n_stages);
        if (i >= p.n_stages) {
            uint32_t par = (uint32_t)(((i / p.n_stages) - 1) & 1);
            if (!wait_bar<0, kHintNs>(smem_base + sm.w_empty + 8 * stage, par, abort_flag, p.status)) { ok = false; break; }
        }
        const int id = (int)(i % slabs);
        const int l = 2 + id / C::PIECES, pc = id % C::PIECES;
        ptx::mbar_expect_tx(smem_base + sm.w_full + 8 * stage, slab);
        // several copies in flight per slab: one large bulk copy did not reach the L2 bandwidth
        for (uint32_t off = 0; off < slab; off += kCopyBytes) {
            const uint32_t bytes = slab - off < kCopyBytes ? slab - off : kCopyBytes;
            ptx::bulk_g2s(smem_base + sm.ring + (uint32_t)stage * slab + off,
                          p.layer[l - 1].qw_umma + (size_t)pc * slab + off, bytes, smem_base + sm.w_full + 8 * stage);
        }
        ++issued;
    }
    if (!ok || *abort_flag) { // let copies in flight land before the CTA may exit
        const unsigned long long t0 = ptx::globaltimer();
        for (long long i = issued > p.n_stages ? issued - p.n_stages : 0; i < issued; ++i) {
            const int stage = (int)(i % p.n_stages);
            const uint32_t par = (uint32_t)((i / p.n_stages) & 1);
            while (!ptx::mbar_try_wait(smem_base + sm.w_full + 8 * stage, par) &&
                   ptx::globaltimer() - t0 < wait_limit_of(abort_flag)) {}
        }
    }
}

// Width 512.  Coordinates: one bulk copy per whole tile (1 KB) into the slot's buffer, issued as
// soon as the slot's threads have taken the previous tile's coordinates out of it.
template <int W, bool SPREAD>
__device__ void xy_role(const FusedParams &p, const SmemMap &sm, uint32_t smem_base, volatile int *abort_flag)
{
    using C = Cfg<W>;
    if (!p.bulk_xy) return;
    uint32_t k[2] = {0, 0};
    bool ok = true;
    for (long long r = 0; ok; ++r) {
        if (tile_index<SPREAD>(r, 0, C::SLOTS) >= p.n_tiles) break;
        for (int s = 0; s < C::SLOTS && ok; ++s) {
            const long long tile = tile_index<SPREAD>(r, s, C::SLOTS);
            if (tile >= p.n_tiles || (tile + 1) * kTile > p.n) continue; // none, or ragged: the threads load it themselves
            if (k[s] > 0 && !wait_bar<0, kHintNs>(smem_base + sm.xy_empty + 8 * s, (k[s] - 1) & 1u, abort_flag, p.status)) { ok = false; break; }
            ptx::mbar_expect_tx(smem_base + sm.xy_full + 8 * s, kTile * 8);
            ptx::bulk_g2s(smem_base + sm.xy + (uint32_t)(s * kTile * 8), p.coords + tile * kTile * 2, kTile * 8, smem_base + sm.xy_full + 8 * s);
            ++k[s];
        }
    }
    if (!ok || *abort_flag) { // let a copy in flight land before the CTA may exit
        const unsigned long long t0 = ptx::globaltimer();
        for (int s = 0; s < C::SLOTS; ++s)
            if (k[s] > 0)
                while (!ptx::mbar_try_wait(smem_base + sm.xy_full + 8 * s, (k[s] - 1) & 1u) && ptx::globaltimer() - t0 < wait_limit_of(abort_flag)) {}
    }
}

template <int W, bool PER_TOKEN, bool ROT, bool SPREAD, bool AHEAD, bool DUMP = false, bool BOTH = false, bool CALIB = false,
          bool GABOR = false, bool MIXED = false>
__global__ void __launch_bounds__(Cfg<W>::THREADS, 1) fused_kernel(const __grid_constant__ ParamsOf<DUMP> p)
{
    using C = Cfg<W>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_u32(smem_raw);
    const uint32_t smem_base = (raw + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - raw);
    const SmemMap sm = smem_map(W, p.n_stages, p.const_words);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem_gen + sm.abort_flag);
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(smem_gen + sm.tmem_holder);

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        *reinterpret_cast<volatile unsigned long long *>(abort_flag + 2) = p.wait_limit_ns;
        for (int i = 0; i < 8; ++i) ptx::mbar_init(smem_base + sm.acc_full + 8 * i, 1);
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(smem_base + sm.acc_last + 8 * s, 1);
            ptx::mbar_init(smem_base + sm.codes_full + 8 * s, C::SLOT_THREADS);
            for (int q = 0; q < 4; ++q) ptx::mbar_init(smem_base + sm.slot_sync + 8 * (s * 4 + q), C::R * 32);
        }
        ptx::mbar_init(smem_base + sm.last_full, 1);
        if constexpr (!C::BULK_XY) {
            for (int s2 = 0; s2 < 2; ++s2) ptx::mbar_init(smem_base + sm.out_sync + 8 * s2, kTile);
        }
        if constexpr (C::BULK_XY) {
            for (int s2 = 0; s2 < 2; ++s2) {
                ptx::mbar_init(smem_base + sm.xy_full + 8 * s2, 1);
                ptx::mbar_init(smem_base + sm.xy_empty + 8 * s2, C::SLOT_THREADS);
            }
        }
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
    // per-layer epilogue constants -> shared memory
    {
        uint32_t *dst = reinterpret_cast<uint32_t *>(smem_gen + sm.consts);
        for (int l = 0; l < p.L - 1; ++l) {
            const FusedLayer &ly = p.layer[l];
            uint32_t *d = dst + ly.c_off;
            const bool fixed = ly.epi_mode == EPI_SINE_FIXED;
            const uint32_t *srcA = fixed ? ly.fxP : reinterpret_cast<const uint32_t *>(ly.cA);
            const uint32_t *srcB = fixed ? ly.fxB : reinterpret_cast<const uint32_t *>(ly.cB);
            const uint32_t *srcC = fixed ? ly.fxQ : reinterpret_cast<const uint32_t *>(ly.cA_lo);
            const int areas = (l == 0) ? (fixed ? 3 : (BOTH ? 5 : 4)) : ((ly.epi_mode == EPI_SINE_WIDE || ly.epi_mode == EPI_SINE_MIXED) ? 3 : 2);
            for (int i = threadIdx.x; i < W; i += C::THREADS) { // i: tensor-memory column, m: its feature
                const int m = fused_feature(i, W);
                d[i] = __ldg(srcA + m);
                d[W + i] = __ldg(srcB + m);
                if (areas >= 3) d[2 * W + i] = __ldg(srcC + m);
                if (areas == 4) d[3 * W + i] = __ldg(ly.qw_k4m + m);
                if (areas == 5) {
                    d[3 * W + i] = (uint32_t)__ldg(ly.l1U + m);
                    d[4 * W + i] = (uint32_t)__ldg(ly.l1V + m);
                }
            }
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    if (warp < kEpiWarps) {
        epilogue_role<W, PER_TOKEN, ROT, SPREAD, AHEAD, DUMP, BOTH, CALIB, GABOR, MIXED>(p, sm, smem_base, warp, lane, tmem_base, abort_flag);
    } else if (warp == kMmaWarp) {
        if (lane == 0) mma_role<W, SPREAD, CALIB>(p, sm, smem_base, tmem_base, abort_flag);
    } else if (warp == kLoadWarp) {
        if (lane == 0) load_role<W, SPREAD, CALIB>(p, sm, smem_base, abort_flag);
        if constexpr (DUMP) {
            // Observing instantiation only (in the timed kernels these few instructions cost 3-4 %): an
            // otherwise idle lane of CTA 0 notes the SM's cycle counter and the global nanosecond timer
            // before the work (status words 2-5); the MMA warp notes them again after it (words 6-9).
            // The ratio of the differences is the SM clock the launch really ran at.
            if (lane == 1 && blockIdx.x == 0) {
                reinterpret_cast<long long *>(p.status)[1] = clock64();
                reinterpret_cast<unsigned long long *>(p.status)[2] = ptx::globaltimer();
            }
        }
    } else {
        if constexpr (C::BULK_XY) {
            if (lane == 0) xy_role<W, SPREAD>(p, sm, smem_base, abort_flag);
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        __syncwarp();
        ptx::tmem_dealloc(tmem_base, 512);
        if constexpr (DUMP) {
            if (lane == 0 && blockIdx.x == 0) {
                reinterpret_cast<long long *>(p.status)[3] = clock64();
                reinterpret_cast<unsigned long long *>(p.status)[4] = ptx::globaltimer();
            }
        }
    }
}

// ------------------------------------------------------------------- choosing an instantiation

typedef void (*fused_fn)(const FusedParams);

template <int W, bool SPREAD, bool AHEAD> fused_fn pick_flags(bool per_token, bool rot)
{
    if (rot) return per_token ? fused_kernel<W, true, true, SPREAD, AHEAD> : fused_kernel<W, false, true, SPREAD, AHEAD>;
    return per_token ? fused_kernel<W, true, false, SPREAD, AHEAD> : fused_kernel<W, false, false, SPREAD, AHEAD>;
}
template <int W, bool AHEAD_OK> fused_fn pick_width(bool per_token, bool rot, bool spread, bool ahead)
{
    if (AHEAD_OK && ahead) return spread ? pick_flags<W, true, AHEAD_OK>(per_token, rot) : pick_flags<W, false, AHEAD_OK>(per_token, rot);
    return spread ? pick_flags<W, true, false>(per_token, rot) : pick_flags<W, false, false>(per_token, rot);
}
typedef void (*fused_dump_fn)(const FusedParamsDump);
// The observing instantiation of a width: the tile mapping and coordinate fetch of the large
// device-memory launches (not spread; fetched ahead where the width has that variant).
template <int W, bool AHEAD_OK> fused_dump_fn pick_dump_width(bool per_token, bool rot)
{
    if (rot) return per_token ? fused_kernel<W, true, true, false, AHEAD_OK, true> : fused_kernel<W, false, true, false, AHEAD_OK, true>;
    return per_token ? fused_kernel<W, true, false, false, AHEAD_OK, true> : fused_kernel<W, false, false, false, AHEAD_OK, true>;
}
// Per-token scales with a layer under EPI_SINE_MIXED: the instantiation that carries the tracked short
// route and its redo (kept out of the others, whose code it would only make larger).  Not spread.
template <int W, bool AHEAD_OK> fused_fn pick_mixed_width(bool rot, bool ahead)
{
    if (AHEAD_OK && ahead) return rot ? fused_kernel<W, true, true, false, AHEAD_OK, false, false, false, false, true>
                                      : fused_kernel<W, true, false, false, AHEAD_OK, false, false, false, false, true>;
    return rot ? fused_kernel<W, true, true, false, false, false, false, false, false, true>
               : fused_kernel<W, true, false, false, false, false, false, false, false, true>;
}
template <int W, bool AHEAD_OK> fused_dump_fn pick_mixed_dump_width(bool rot)
{
    return rot ? fused_kernel<W, true, true, false, AHEAD_OK, true, false, false, false, true>
               : fused_kernel<W, true, false, false, AHEAD_OK, true, false, false, false, true>;
}
// The two-sided transform's kernels: not spread, coordinates not fetched ahead.
template <int W> fused_fn pick_both_width(bool per_token)
{
    return per_token ? fused_kernel<W, true, true, false, false, false, true> : fused_kernel<W, false, true, false, false, false, true>;
}
template <int W> fused_dump_fn pick_both_dump_width(bool per_token)
{
    return per_token ? fused_kernel<W, true, true, false, false, true, true> : fused_kernel<W, false, true, false, false, true, true>;
}
// Calibration kernels (per-tensor activation scales): the network up to the rotated input of layer
// p.L, whose absmax they take.
template <int W> fused_fn pick_calib_width(bool rot, bool gabor, bool both)
{
    if (both) return gabor ? fused_kernel<W, false, true, false, false, false, true, true, true> : fused_kernel<W, false, true, false, false, false, true, true, false>;
    if (gabor) return rot ? fused_kernel<W, false, true, false, false, false, false, true, true> : fused_kernel<W, false, false, false, false, false, false, true, true>;
    return rot ? fused_kernel<W, false, true, false, false, false, false, true> : fused_kernel<W, false, false, false, false, false, false, true>;
}
// The wavelet activation's kernels: not spread, coordinates not fetched ahead.
template <int W> fused_fn pick_gabor_width(bool per_token, bool rot)
{
    if (rot) return per_token ? fused_kernel<W, true, true, false, false, false, false, false, true>
                              : fused_kernel<W, false, true, false, false, false, false, false, true>;
    return per_token ? fused_kernel<W, true, false, false, false, false, false, false, true>
                     : fused_kernel<W, false, false, false, false, false, false, false, true>;
}
// The wavelet activation with the two-sided transform.
template <int W> fused_fn pick_gabor_both_width(bool per_token)
{
    return per_token ? fused_kernel<W, true, true, false, false, false, true, false, true> : fused_kernel<W, false, true, false, false, false, true, false, true>;
}
template <int W> fused_dump_fn pick_gabor_both_dump_width(bool per_token)
{
    return per_token ? fused_kernel<W, true, true, false, false, true, true, false, true> : fused_kernel<W, false, true, false, false, true, true, false, true>;
}
template <int W> fused_dump_fn pick_gabor_dump_width(bool per_token, bool rot)
{
    if (rot) return per_token ? fused_kernel<W, true, true, false, false, true, false, false, true>
                              : fused_kernel<W, false, true, false, false, true, false, false, true>;
    return per_token ? fused_kernel<W, true, false, false, false, true, false, false, true>
                     : fused_kernel<W, false, false, false, false, true, false, false, true>;
}
// One translation unit per width (dhq_fused_w*.cu) instantiates the kernels of that width.
fused_fn fused_pick_64(bool per_token, bool rot, bool spread, bool ahead);
fused_fn fused_pick_128(bool per_token, bool rot, bool spread, bool ahead);
fused_fn fused_pick_256(bool per_token, bool rot, bool spread, bool ahead);
fused_fn fused_pick_512(bool per_token, bool rot, bool spread, bool ahead);
fused_dump_fn fused_pick_dump_64(bool per_token, bool rot);
fused_dump_fn fused_pick_dump_128(bool per_token, bool rot);
fused_dump_fn fused_pick_dump_256(bool per_token, bool rot);
fused_dump_fn fused_pick_dump_512(bool per_token, bool rot);
fused_fn fused_pick_gabor_64(bool per_token, bool rot);
fused_fn fused_pick_gabor_128(bool per_token, bool rot);
fused_fn fused_pick_gabor_256(bool per_token, bool rot);
fused_fn fused_pick_gabor_512(bool per_token, bool rot);
fused_fn fused_pick_mixed_64(bool rot, bool ahead);
fused_fn fused_pick_mixed_128(bool rot, bool ahead);
fused_fn fused_pick_mixed_256(bool rot, bool ahead);
fused_fn fused_pick_mixed_512(bool rot, bool ahead);
fused_dump_fn fused_pick_mixed_dump_64(bool rot);
fused_dump_fn fused_pick_mixed_dump_128(bool rot);
fused_dump_fn fused_pick_mixed_dump_256(bool rot);
fused_dump_fn fused_pick_mixed_dump_512(bool rot);
fused_fn fused_pick_gabor_both_64(bool per_token);
fused_fn fused_pick_gabor_both_128(bool per_token);
fused_fn fused_pick_gabor_both_256(bool per_token);
fused_fn fused_pick_gabor_both_512(bool per_token);
fused_dump_fn fused_pick_gabor_both_dump_64(bool per_token);
fused_dump_fn fused_pick_gabor_both_dump_128(bool per_token);
fused_dump_fn fused_pick_gabor_both_dump_256(bool per_token);
fused_dump_fn fused_pick_gabor_both_dump_512(bool per_token);
fused_dump_fn fused_pick_gabor_dump_64(bool per_token, bool rot);
fused_dump_fn fused_pick_gabor_dump_128(bool per_token, bool rot);
fused_dump_fn fused_pick_gabor_dump_256(bool per_token, bool rot);
fused_dump_fn fused_pick_gabor_dump_512(bool per_token, bool rot);
fused_fn fused_pick_calib_64(bool rot, bool gabor, bool both);
fused_fn fused_pick_calib_128(bool rot, bool gabor, bool both);
fused_fn fused_pick_calib_256(bool rot, bool gabor, bool both);
fused_fn fused_pick_calib_512(bool rot, bool gabor, bool both);
fused_fn fused_pick_both_64(bool per_token);
fused_fn fused_pick_both_128(bool per_token);
fused_fn fused_pick_both_256(bool per_token);
fused_fn fused_pick_both_512(bool per_token);
fused_dump_fn fused_pick_both_dump_64(bool per_token);
fused_dump_fn fused_pick_both_dump_128(bool per_token);
fused_dump_fn fused_pick_both_dump_256(bool per_token);
fused_dump_fn fused_pick_both_dump_512(bool per_token);

} // namespace dhq
