/*
 * dhq_peaks.h - micro-benchmarks of the execution pipes that bound the DHQ forward kernel.
 *
 * The paper (arXiv 2508.13478) has no counterpart: its cost model is FPGA resources (Table 2).
 * On a GPU the same datapath (Section III-C: MAC array, activation, dynamic quantization) is
 * bounded by the int8 tensor pipe, the special-function unit (sine) and the plain fp32/integer
 * pipes, whose peaks these loops measure so that roofline fractions have measured denominators.
 */
#ifndef DHQ_PEAKS_H_
#define DHQ_PEAKS_H_

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define DHQ_PEAKS_API
#else
#define DHQ_PEAKS_API __attribute__((visibility("default")))
#endif

typedef enum {
    DHQ_PIPE_FFMA = 0,     /* fp32 fused multiply-add, independent chains          */
    DHQ_PIPE_FADD = 1,     /* fp32 add                                             */
    DHQ_PIPE_MUFU_SIN = 2, /* sin.approx.f32 (multiply by 1/2pi + special function) */
    DHQ_PIPE_I2F = 3,      /* cvt.rn.f32.s32                                       */
    DHQ_PIPE_F2I = 4,      /* cvt.rni.s32.f32                                      */
    DHQ_PIPE_PRMT = 5,     /* byte permute                                         */
    DHQ_PIPE_FMNMX = 6,    /* fp32 min/max                                         */
    DHQ_PIPE_TENSOR_I8 = 7, /* tcgen05.mma kind::i8, 128x256x32, operands resident in shared memory */
    DHQ_PIPE_FADD2 = 8,    /* add.rn.f32x2: two fp32 adds per lane and instruction (counted as 2)   */
    DHQ_PIPE_FFMA2 = 9,    /* fma.rn.f32x2 (counted as 2)                                            */
    /* The fused kernel's own per-element loops for a hidden layer of width 256, run alone (16 warps per
     * SM, data in tensor memory, no MMA, no barrier, no tile loop); counted in activation elements:    */
    DHQ_PIPE_PASS1 = 10,   /* dequantize + bias + sine + butterfly stages with stride < 64             */
    DHQ_PIPE_PASS2 = 11,   /* butterfly stages 64 and 128 + quantizer + code stores to shared memory   */
    DHQ_PIPE_PASS12 = 12   /* both, one after the other                                                */
} dhq_pipe_t;

/*
 * Runs one micro-benchmark on the current device (all SMs busy), timed with CUDA events on
 * `stream` after one warm-up launch; synchronizes.
 *   ops_per_s  host, receives operations per second: instructions x 32 lanes for the scalar
 *              pipes (an FMA counts as one), 2*M*N*K integer operations per MMA for the tensor
 *              pipe, activation elements for the PASS loops.
 *   ms         host, receives the duration of the timed launch, or NULL.
 * Returns 0 on success, a negative value on a CUDA error or unknown pipe, 1 if the tensor-pipe
 * loop hit its bounded wait.
 */
DHQ_PEAKS_API int dhq_measure_pipe(int pipe, int iters, void *stream, double *ops_per_s, double *ms);

/*
 * Accuracy of the sine the epilogue uses (the activation of Section III-C's input and linear
 * layers), measured on the current device: the largest |f(x) - sin(x)| over `count` fp32
 * arguments spread evenly over [lo, hi], against the fp64 sine of the same argument.
 *   mode 0: the hardware approximation sin.approx.f32 alone (what the fast epilogue applies to
 *           phases below its limit); mode 1: with the explicit two-part 2 pi reduction in front
 *           (the wide epilogue).
 * The fast epilogue's phase limit follows from this curve and the 1e-5 output tolerance.
 * Synchronizes `stream`.  Returns 0, or a negative value on bad arguments or a CUDA error.
 */
DHQ_PEAKS_API int dhq_measure_sine_error(float lo, float hi, long long count, int mode, void *stream,
                                         double *max_abs_err);

#ifdef __cplusplus
}
#endif
#endif /* DHQ_PEAKS_H_ */
