// Per-element arithmetic shared by every kernel of the library, so that the layer-by-layer
// path and the fused path execute the same fp32 operations in the same order and agree bit
// for bit.  Every fp32 step uses an explicit round-to-nearest intrinsic: nothing here may be
// contracted, reassociated or replaced by a fast-math variant.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace dhq {

// Epilogue variants, chosen per layer when the network is prepared.
enum EpiMode : int {
    EPI_LINEAR = 0,    // last layer: z = c * acc + b
    EPI_SINE_FAST = 1, // hidden layer whose phase stays below kFastPhaseLimit (bound taken at prepare time over all
                       // unsaturated inputs, quantization error of weights and activations included): sin.approx(fma(acc, c, B))
    EPI_SINE_WIDE = 2, // large phases: compensated phase and explicit 2*pi reduction
    EPI_SINE_FIXED = 3, // first layer with a per-tensor activation scale: phase in 32-bit fixed point
    EPI_BOTH = 4,      // two-sided transform: the layer kernel undoes the output-side rotation in fp64
    EPI_SINE_MIXED = 5 // hidden layer without a bound below the limit: decided per value, x = fma(acc, c, B);
                       // |x| <= limit -> sin.approx(x), else the compensated phase and explicit reduction
};

// Largest |omega0 z| for which EPI_SINE_FAST keeps the result within 1e-5 of an exact sine.  Worst
// case at the limit, term by term: rounding of the fma result (half an ulp of a value in [32, 64):
// 1.9e-6), rounding of the constant c to fp32 (36 * 2^-24 = 2.1e-6) and of B (1e-7), and the
// hardware approximation itself, measured on B200 against the fp64 sine over 2^24 arguments per
// range (dhq_measure_sine_error): 6.2e-7 for |x| <= 3.2, 2.3e-6 to 16, 4.4e-6 to 32, 4.6e-6 to 40,
// 5.0e-6 to 48, 8.3e-6 to 56 - its internal multiply by 1/(2 pi) loses absolute accuracy as the
// argument grows.  Sum at 36: 8.7e-6.  With a per-token activation scale the constant is the product
// fl32(cA * s_x) of two rounded factors (twice the constant error) and the limit is 32 rad, where the
// fma result still has half the ulp: 0.95e-6 + 3.8e-6 + 1e-7 + 4.4e-6 = 9.3e-6.
constexpr float kFastPhaseLimit = 36.0f;
constexpr float kFastPhaseLimitPerToken = 32.0f;
// Two-sided transform inside the fused kernel: acc' = H_M acc may pass 2^24, so its conversion to
// fp32 adds a relative 2^-24 to the phase; with the limit at 24 rad the sum is 0.95e-6 (fma) + 2.9e-6
// (constant, twice for a per-token scale) + 1.4e-6 (conversion) + 4.4e-6 (approximation) = 9.7e-6.
constexpr float kMixedPhaseLimitBoth = 24.0f;

__device__ __forceinline__ float qmax_of(int bits) { return (float)((1 << (bits - 1)) - 1); }

// Symmetric absmax scales: s = a / qmax, inv = qmax / a, both IEEE divisions; a = 0 -> 0, 0.
// An absmax so small that qmax / a is not a finite fp32 number (a below about 3.7e-37 at 8 bits)
// counts as zero: no code can be formed with an infinite scale, and values of that size
// contribute nothing.
__device__ __forceinline__ void scales_of(float a, float qmaxf, float &s, float &inv)
{
    const float s_ = __fdiv_rn(a, qmaxf), i_ = __fdiv_rn(qmaxf, a);
    const bool ok = a > 0.0f && i_ <= 3.402823466e+38f; // false for a = 0 (i_ = inf), NaN, and the overflow case
    s = ok ? s_ : 0.0f;
    inv = ok ? i_ : 0.0f;
}

// q = clamp(round_half_even(fl32(v * inv)), -qmax, +qmax).  Clamping before rounding gives the
// same integer because qmax is one.  NaN inputs come out as +-qmax (fminf/fmaxf drop the NaN).
__device__ __forceinline__ int quantize(float v, float inv, float qmaxf)
{
    float t = __fmul_rn(v, inv);
    t = fmaxf(fminf(t, qmaxf), -qmaxf);
    return __float2int_rn(t);
}

__device__ __forceinline__ float sin_approx(float x)
{
    float y;
    asm("sin.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// sin(x) for |x| up to a few thousand: k = nearest integer to x / (2 pi), r = x - k * 2 pi with
// 2 pi split into fl32(2 pi) and the remainder (two fused multiply-adds, each exact before its
// single rounding), then the hardware approximation on |r| <= pi.
__device__ __forceinline__ float sin_wide(float x)
{
    const float inv_two_pi = 0.15915494309189535f;
    const float two_pi_hi = 6.2831854820251465f;   // fl32(2 pi)
    const float two_pi_lo = -1.7484555e-07f;       // 2 pi - fl32(2 pi)
    // nearest integer by adding and subtracting 1.5 * 2^23 (ties to even; |x / 2 pi| < 2^22)
    float k = __fsub_rn(__fadd_rn(__fmul_rn(x, inv_two_pi), 12582912.0f), 12582912.0f);
    float r = __fmaf_rn(k, -two_pi_hi, x);
    r = __fmaf_rn(k, -two_pi_lo, r);
    return sin_approx(r);
}

// Per-(token, channel) epilogue.  accf = (float)acc is exact (|acc| < 2^24).
//   c_hi, c_lo : the dequantization constant omega0 * s_w * s_x (or s_w * s_x for the last
//                layer) as an fp32 value and its remainder; c_lo is only read by EPI_SINE_WIDE.
//   cb         : omega0 * b (or b for the last layer).
__device__ __forceinline__ float epilogue(int mode, float accf, float c_hi, float c_lo, float cb)
{
    if (mode == EPI_SINE_FAST) return sin_approx(__fmaf_rn(accf, c_hi, cb));
    if (mode == EPI_SINE_WIDE) return sin_wide(__fmaf_rn(accf, c_lo, __fmaf_rn(accf, c_hi, cb)));
    return __fmaf_rn(accf, c_hi, cb);
}

// EPI_SINE_MIXED: the rule is per value and depends on nothing but (acc, constants), so every kernel
// that applies it gives the same bits.  The error terms listed at kFastPhaseLimit all grow with the
// phase that is actually computed, so a value below the limit is as accurate as under EPI_SINE_FAST.
__device__ __forceinline__ float epilogue_mixed(float accf, float c_hi, float c_lo, float cb, float limit)
{
    const float x = __fmaf_rn(accf, c_hi, cb);
    if (fabsf(x) <= limit) return sin_approx(x);
    return sin_wide(__fmaf_rn(accf, c_lo, x));
}

// Wavelet activation (reading of the paper's WIRE experiments, Section IV): the real Gabor wavelet
// psi(z) = sin(omega0 z) exp(-(s0 z)^2), from the compensated phase x = omega0 z and c = s0 / omega0.
// The envelope's exponent carries a relative error of a few 2^-24, the result stays within the
// sine's own error.
__device__ __forceinline__ float gabor_epilogue(float accf, float c_hi, float c_lo, float cb, float c)
{
    const float x = __fmaf_rn(accf, c_lo, __fmaf_rn(accf, c_hi, cb));
    const float g = __fmul_rn(x, c);
    float e;
    asm("ex2.approx.f32 %0, %1;" : "=f"(e) : "f"(__fmul_rn(__fmul_rn(g, g), -1.4426950408889634f)));
    return __fmul_rn(sin_wide(x), e);
}

// First layer, per-tensor activation scale.  The rotated padded coordinate [x, y, 0, 0] has the
// codes [qs, qd, qs, qd], so acc[m] = qs * u_m + qd * v_m with u_m = q_w[m][0] + q_w[m][2],
// v_m = q_w[m][1] + q_w[m][3].  With P = frac(c u_m / 2 pi), Q = frac(c v_m / 2 pi),
// B = frac(omega0 b_m / 2 pi) held as 32-bit binary fractions of a turn (c = omega0 s_w s_x), the
// phase in turns is qs * P + qd * Q + B modulo 1: unsigned 32-bit arithmetic wraps exactly where
// the sine is periodic, so no range reduction is needed and the error is that of the constants
// (at most 127 * 2^-33 turns each) plus one int->float rounding (2^-26 turns).
__device__ __forceinline__ float sine_fixed(int qs, int qd, uint32_t P, uint32_t Q, uint32_t B)
{
    uint32_t ph = (uint32_t)qs * P + ((uint32_t)qd * Q + B);
    return sin_approx(__fmul_rn((float)(int)ph, 1.4629180792671596e-09f)); // 2 pi / 2^32
}

// Per-token activation scales: the per-channel constant cA (+ remainder cA_lo) times the
// token's s_x.  c_lo collects the rounding error of that product and the remainder term.
__device__ __forceinline__ void token_const(float cA, float cA_lo, float s_x, float &c_hi, float &c_lo)
{
    c_hi = __fmul_rn(cA, s_x);
    c_lo = __fmaf_rn(cA_lo, s_x, __fmaf_rn(cA, s_x, -c_hi));
}

} // namespace dhq
