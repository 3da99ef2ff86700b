/*
 * dhq.h - C ABI of the B200 library for the fully quantized forward pass of a sinusoidal INR
 * (DHQ, arXiv 2508.13478).
 *
 * The network is f_theta : coordinate -> signal value (Section II-A of the paper), an MLP with L
 * linear layers of sizes dims[0] = 2, dims[1..L-1] = w, dims[L] in 1..4.  Every layer l computes
 * (Section III-B and III-C):
 *
 *     x~   = H_K x_l                      online Walsh-Hadamard rotation of the layer input (Eq. 3)
 *     q_x  = Q_a(x~)                      activation quantizer ("dynamic quantization module")
 *     acc  = q_x * q_W^T                  integer matmul, int32 accumulation, on the tensor cores
 *     z    = s_W s_x acc + b              dequantize and add the bias
 *     x_{l+1} = sin(omega0 z)             hidden layers; the last layer returns z (no activation)
 *
 * with q_W = Q_w(W H_K / K) prepared once (Eq. 4-5, the factor acting on the input dimension;
 * H is symmetric, so (W H/K)(H x) = W x).  The 2 inputs are zero-padded to K = 4 and the outputs
 * of the last layer to 4, so every Hadamard size is a power of two.
 *
 * Quantizer Q (one quantizer for all layers, Section III-B), as implemented: symmetric,
 * qmax = 2^(bits-1) - 1, a = max |v| over the tensor / output channel / token,
 * s = a / qmax and inv = qmax / a in IEEE fp32, q = clamp(round_half_even(fl32(v * inv)), +-qmax),
 * a = 0 gives s = inv = 0 and all-zero codes.  Codes of every bit-width live in int8 lanes.
 * The fp32 rotation adds in the order of the in-place butterfly with strides 1, 2, 4, ..., K/2,
 * where the pair (i, i+h) becomes (a+b, a-b); outputs are in natural (Sylvester) order.
 *
 * Conventions for every call:
 *   - Pointers named "device" are CUDA device pointers owned by the caller; the library never
 *     frees them and does not keep them after the call's stream work has run.  "host" pointers are
 *     ordinary host memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Work is enqueued
 *     on it and the call returns without waiting, unless stated otherwise.
 *   - Argument errors are reported by the return value and enqueue nothing.  Conditions found on
 *     the device (a bounded wait that ran out) are recorded in a status word read by
 *     dhq_last_status.  Nothing traps, aborts or throws.
 *   - With the environment variable DHQ_LOG set (to anything but "0") dhq_prepare, dhq_calibrate,
 *     dhq_forward and dhq_forward_host write one line per call to stderr (size, shape, route, status,
 *     kernels enqueued).
 *   - One forward may be in flight per handle at a time.  Handles belong to the device that was
 *     current in dhq_prepare; that device must be current in later calls (INVALID_ARG otherwise).
 */
#ifndef DHQ_H_
#define DHQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define DHQ_API
#else
#define DHQ_API __attribute__((visibility("default")))
#endif

typedef struct dhq_handle_s *dhq_handle_t; /* opaque, owned by the library */

typedef enum {
    DHQ_OK = 0,
    DHQ_ERR_INVALID_ARG = 1,    /* NULL pointer, negative size, malformed config           */
    DHQ_ERR_UNSUPPORTED = 2,    /* shape or option outside what the kernels implement      */
    DHQ_ERR_ALLOC = 3,          /* device or host allocation failed                        */
    DHQ_ERR_CUDA = 4,           /* a CUDA runtime call failed                              */
    DHQ_ERR_NOT_CALIBRATED = 5, /* per-tensor activation scales requested but not frozen   */
    DHQ_ERR_TIMEOUT = 6,        /* a bounded wait inside a kernel ran out                  */
    DHQ_ERR_TOO_LARGE = 7       /* more tokens than a fixed-size scratch area can hold     */
} dhq_status_t;

/* Quantizer granularity: weights per tensor or per output channel; activations per tensor
 * (static: frozen by calibration) or per token (dynamic: from each coordinate's own values). */
typedef enum { DHQ_GRAN_TENSOR = 0, DHQ_GRAN_CHANNEL_OR_TOKEN = 1 } dhq_gran_t;

/* Which side of Eq. 4 is applied.  DHQ_ROT_INPUT is the DHQ path; DHQ_ROT_NONE skips the rotation
 * of weights and activations (the plain uniform quantizer the paper compares against, Section
 * IV-B) with everything else unchanged.  DHQ_ROT_BOTH is Eq. 4-5 taken literally, W~ = H_M W H_K /
 * (K M) (rows first, then columns, same fp32 butterfly order), with the layer output
 * z = H_M (s_w s_x acc) + b: the output-side rotation is undone after the integer product and
 * before the bias.  With one weight scale per tensor (w_gran = DHQ_GRAN_TENSOR) it runs inside
 * the fused kernel: H_M is applied to the int32 accumulators, exactly (the library checks at
 * prepare time that qmax_a * sum |q_w| < 2^31, so nothing can overflow), then the fp32 epilogue;
 * about 1.6-1.7 times the time of DHQ_ROT_INPUT.  With per-output-channel weight scales the
 * rotation has to act on the dequantized values; that case runs layer by layer (one kernel pass
 * per layer, fp64 rotation), as does dhq_forward_debug for either.  Both routes are within 1e-5 of
 * the definition; they are not bit-identical to each other (fp32 against fp64 epilogue), so for
 * DHQ_ROT_BOTH dhq_forward and dhq_forward_debug need not agree bit for bit;
 * dhq_forward_fused_debug observes the fused route.  dhq_forward_static_scratch does not take it. */
typedef enum { DHQ_ROT_INPUT = 0, DHQ_ROT_BOTH = 1, DHQ_ROT_NONE = 2 } dhq_rot_t;

/* Bit-width value that means "not quantized, fp32": the comparison datapaths of the paper's
 * motivation figure (Section I) and hardware table (Table 2).
 *   w_bits 2..8, a_bits 2..8            the fully quantized network (W8A8 and the narrower sweeps)
 *   w_bits 2..8, a_bits DHQ_BITS_FLOAT  W8A32: weights folded and quantized as above, activations
 *                                       kept in fp32 (rotated in fp32 when rotation = DHQ_ROT_INPUT):
 *                                       z = s_w sum_k q_w x~_k + b
 *   both DHQ_BITS_FLOAT                 W32A32: the plain fp32 network, z = W x + b (rotation ignored)
 * The two floating-point datapaths run one kernel pass per layer with fp32 multiply-adds on the
 * CUDA cores (activations in device memory between layers).  They need no calibration; the
 * calibration calls are no-ops for them.  dhq_forward_debug dumps only X and Y for them;
 * dhq_forward_fused_debug, dhq_forward_static_scratch and DHQ_ROT_BOTH are UNSUPPORTED.
 * Their layer outputs carry fp32 summation and phase rounding error: they are checked against the
 * fp64 definition within 2e-5 per layer (measured: 5.6e-6), not 1e-5. */
#define DHQ_BITS_FLOAT 32

/* Activation of layers 1..L-1.  DHQ_ACT_SINE: sin(omega0 z), the SIREN of the paper's method
 * sections.  DHQ_ACT_GABOR: the real Gabor wavelet sin(omega0 z) exp(-(act_s0 z)^2), this
 * library's reading of the "wavelet activation" of the WIRE experiments (Section IV; the paper
 * gives no formula, the complex form of the WIRE paper is not built).  dhq_forward runs it inside
 * the fused kernel (an instantiation whose epilogue multiplies the sine by the envelope; same
 * arithmetic as the layer-by-layer kernel, so dhq_forward_debug agrees with it bit for bit);
 * dhq_forward_fused_debug observes that instantiation's per-layer values; DHQ_ROT_BOTH combines
 * with it under the same rule as for the sine (fused with one weight scale per tensor, else
 * layer by layer).  It needs omega0 != 0; the floating-point datapaths and
 * dhq_forward_static_scratch do not take it. */
typedef enum { DHQ_ACT_SINE = 0, DHQ_ACT_GABOR = 1 } dhq_act_t;

typedef struct {
    int n_layers;       /* L linear layers, 2..16                                          */
    const int *dims;    /* host, L+1 ints: 2, w, ..., w, d_L; w a power of two in 64..512, */
                        /* the same for all hidden layers; d_L in 1..4                     */
    int w_bits, a_bits; /* 2..8, or DHQ_BITS_FLOAT (see above)                             */
    float omega0;       /* sine frequency of layers 1..L-1                                 */
    dhq_gran_t w_gran;
    dhq_gran_t a_gran;
    dhq_rot_t rotation; /* DHQ_ROT_INPUT, DHQ_ROT_NONE or DHQ_ROT_BOTH                     */
    dhq_act_t activation; /* DHQ_ACT_SINE or DHQ_ACT_GABOR                                 */
    float act_s0;       /* width parameter of the Gabor wavelet (> 0); ignored for the sine */
} dhq_config_t;

/*
 * Per-layer dump targets for dhq_forward_debug.  Each member is a host array of L device
 * pointers (entry l-1 for layer l); a NULL member or NULL entry is skipped.  K and M are the
 * padded sizes of the layer as the definition pads them: K = 4 for layer 1, else w; M = 4 for
 * layer L, else w.
 */
typedef struct {
    float **X;      /* [n][K] fp32   layer input (layer 1: [x, y, 0, 0])                   */
    int8_t **codes; /* [n][K] int8   quantized rotated input                               */
    float **s_x;    /* [n]    fp32   activation scale of each token                        */
    int32_t **acc;  /* [n][M] int32  integer accumulators                                  */
    float **Y;      /* [n][M] fp32   layer output (after the sine for hidden layers)       */
} dhq_debug_bufs_t;

/*
 * Weight side, once per network (Eq. 4-5 and the quantizer of Section III-B), run on the
 * device: pad, rotate every row by H_K in fp32, scale by the exact 1/K, quantize, and pack the
 * codes into the shared-memory image the tensor-core kernel loads.
 *   cfg    host.
 *   W      host array of L device pointers; W[l-1] is row-major [dims[l]][dims[l-1]] fp32
 *          (the layout of a PyTorch nn.Linear weight).
 *   b      host array of L device pointers; b[l-1] is [dims[l]] fp32.
 *   out    receives the handle.  The caller releases it with dhq_destroy.
 * Allocates device memory; enqueues the preparation kernels on `stream` and returns.  W and b
 * may be released once that stream work has completed.
 * Errors: INVALID_ARG (NULL, n_layers out of range), UNSUPPORTED (dims[0] != 2, width not a
 * power of two in 64..512 or not uniform, d_L outside 1..4, a bit-width combination other than
 * those listed at DHQ_BITS_FLOAT, unknown rotation or activation), ALLOC, CUDA.
 */
DHQ_API dhq_status_t dhq_prepare(const dhq_config_t *cfg, const float *const *W,
                                 const float *const *b, void *stream, dhq_handle_t *out);

/*
 * Freeze the per-tensor activation scales (a_gran = DHQ_GRAN_TENSOR) on a set of coordinates:
 * for l = 1..L, a_l = max over the n tokens and the K features of |H_K x_l|, taken with layers
 * < l already quantized with their frozen scales (the run-time statistic of the "dynamic
 * quantization module", Section III-C, taken once and kept, so that a coordinate's output does
 * not depend on the batch it arrives in).
 *   coords device [n][2] fp32, n >= 1.
 * Enqueues L passes on `stream` (one launch of the fused kernel per layer, run up to that layer's
 * rotated input; layer-by-layer kernels for handles without a fused kernel).  With a_gran = per
 * token the call is a no-op returning DHQ_OK.
 * Errors: INVALID_ARG, ALLOC, CUDA.
 */
DHQ_API dhq_status_t dhq_calibrate(dhq_handle_t h, const float *coords, int64_t n, void *stream);

/*
 * The same calibration one layer at a time, for coordinate sets that are spread over several
 * GPUs (coordinates are independent, Section III: f_theta maps each x to its y; each GPU holds a
 * replica of the handle and a part of the set).  The frozen value of layer l is the maximum over
 * ALL parts, and layer l+1 may only be measured once layer l is frozen, so the caller alternates,
 * for l = 1..L:
 *   dhq_calibrate_layer(h, l, part, n_part, stream)   measure this part: max |H_K x_l| into the handle;
 *   dhq_get_act_absmax(h, l, &a, stream)              read it (synchronizes the stream);
 *   a = maximum of a over the parts                   (one float: an all-reduce(max), or a host loop);
 *   dhq_set_act_absmax(h, l, a, stream)               freeze layer l: scales and epilogue constants.
 * After layer L the handle is calibrated exactly as by dhq_calibrate on the whole set (the
 * maximum of non-negative floats does not depend on how the set was split).  n_part = 0 is
 * allowed and contributes 0.  dhq_calibrate_layer(l) needs layers < l frozen (by this sequence or
 * an earlier calibration): otherwise NOT_CALIBRATED.  Starting the sequence marks the handle as
 * not calibrated until layer L is set.  With per-token activation scales all three are no-ops
 * (dhq_get_act_absmax then returns whatever the handle holds).
 *   absmax  host pointer (get) / finite value >= 0 (set).
 * Errors: INVALID_ARG, NOT_CALIBRATED, ALLOC, CUDA.
 */
DHQ_API dhq_status_t dhq_calibrate_layer(dhq_handle_t h, int layer, const float *coords, int64_t n,
                                         void *stream);
DHQ_API dhq_status_t dhq_get_act_absmax(dhq_handle_t h, int layer, float *absmax, void *stream);
DHQ_API dhq_status_t dhq_set_act_absmax(dhq_handle_t h, int layer, float absmax, void *stream);

/*
 * The forward pass f_theta over n coordinates: one launch of the fused kernel, activations
 * never leave the SM between layers.
 *   coords device [n][2] fp32 (x, y per token), 8-byte aligned.
 *   out    device [n][d_L] fp32, dense.
 * n = 0 is a no-op; n need not be a multiple of any tile size.  If the handle uses per-tensor
 * activation scales and none are frozen yet, this call first calibrates on its own coordinates
 * (as dhq_calibrate) and freezes them; later calls reuse them.
 * Non-finite coordinates give unspecified values but do not hang.
 * Accuracy: every layer's fp32 output is within 1e-5 of the definition evaluated in fp64 on the
 * same codes as long as the layer's phases |omega0 z| stay below 256 rad (the paper's networks
 * and the SIREN initialisation stay below about 50); beyond that the fp32 phase itself carries half
 * an ulp, 1.5e-5 rad at 256..512 rad and twice that per further doubling.
 * On a handle with a fused kernel and frozen (or per-token) scales the call enqueues that one
 * launch and nothing else - no allocation, no synchronisation - so it may be recorded by stream
 * capture into a CUDA graph and replayed on new contents of the same buffers.
 * Errors: INVALID_ARG, ALLOC, CUDA.
 */
DHQ_API dhq_status_t dhq_forward(dhq_handle_t h, const float *coords, int64_t n, float *out,
                                 void *stream);

/*
 * As dhq_forward but with HOST buffers.  The call is ordered after earlier work on `stream`, and
 * later work on `stream` waits for the result to be in out_host.
 *   - Both buffers pinned (page-locked, e.g. cudaHostAlloc / cudaHostRegister) and the scales
 *     already frozen: no staging and no copy call.  The fused kernel reads the coordinates and
 *     writes the result through the buffers' device mapping, so the transfers over the host link
 *     happen tile by tile inside the one launch, beside the arithmetic (with out_host 16-byte
 *     aligned, each whole tile of results leaves by one bulk store).
 *   - Otherwise (pageable memory, or the first per-tensor call, which calibrates): the data is
 *     staged in device buffers owned by the handle, grown on demand (this may allocate and
 *     synchronize the first time a larger n is seen).  Larger n is cut into up to 8 launches, each
 *     a whole number of tile rounds of the fused kernel, whose copies run on two streams owned
 *     by the handle beside the kernels (streams and events are created on the first such call).
 * Results do not depend on the route or the cut.  If a device-side wait times out in one launch,
 * later launches of the same call still run; the status word read by dhq_last_status records it.
 */
DHQ_API dhq_status_t dhq_forward_host(dhq_handle_t h, const float *coords_host, int64_t n,
                                      float *out_host, void *stream);

/*
 * Layer-by-layer forward that writes every intermediate to the caller's buffers (see
 * dhq_debug_bufs_t), for checking each stage against a reference.  Same arithmetic as
 * dhq_forward, operation for operation, so `out` and Y[L-1] equal dhq_forward's output bit for
 * bit; activations go through device memory between layers, in chunks, using scratch memory
 * owned by the handle.  `out` and `bufs` may each be NULL.  Requires frozen scales when
 * a_gran = per tensor (NOT_CALIBRATED otherwise).
 */
DHQ_API dhq_status_t dhq_forward_debug(dhq_handle_t h, const float *coords, int64_t n, float *out,
                                       const dhq_debug_bufs_t *bufs, void *stream);

/*
 * The forward pass by the fused kernel itself, observed: the same kernel as dhq_forward (one
 * launch, tensor-core products, activations staying on the SM; Section III-C's dataflow) compiled
 * with stores added at the places where each per-layer value exists - the codes as they go into
 * the tensor-core operand tile, the activation scale, the int32 accumulators as they are read
 * from tensor memory, the layer output after the sine.  Same arithmetic, instruction for
 * instruction, so `out` equals dhq_forward's bit for bit; it runs slower because of the stores.
 *   bufs   as for dhq_forward_debug.  Inside the fused kernel the input of layer l+1 is the output
 *          of layer l (one value): X[l] receives a copy of Y[l-1].  The first layer's accumulators
 *          are never formed on the per-tensor route (its phase is built from the two distinct
 *          input codes); acc[0] holds codes . weight codes computed for the dump.
 *          X[0] must be 16-byte aligned, the other buffers 4-byte aligned.
 * Requires frozen scales when a_gran = per tensor (NOT_CALIBRATED otherwise).  A handle that runs
 * layer by layer (DHQ_ROT_BOTH with per-channel weight scales, the
 * floating-point datapaths) is observed by dhq_forward_debug: UNSUPPORTED here.
 * Errors: INVALID_ARG, UNSUPPORTED, NOT_CALIBRATED, CUDA.
 */
DHQ_API dhq_status_t dhq_forward_fused_debug(dhq_handle_t h, const float *coords, int64_t n, float *out,
                                             const dhq_debug_bufs_t *bufs, void *stream);

/*
 * Bound of the waits inside the fused kernel.  Its warps hand tiles to each other through
 * barriers in shared memory; every such wait gives up after this long, the kernel then records
 * DHQ_ERR_TIMEOUT in the handle's status word (dhq_last_status), releases what it holds and
 * returns, so that a stall never holds the GPU.  Default 2 s; at least 1000 ns.  Takes effect
 * with the next launch.  (The paper's pipeline has no counterpart: an FPGA pipeline cannot
 * stall this way.)
 */
DHQ_API dhq_status_t dhq_set_wait_limit(dhq_handle_t h, int64_t nanoseconds);

/*
 * Test hook for that bound: the next fused-kernel launch of this handle (dhq_forward or the
 * pinned route of dhq_forward_host) leaves out the copy of the last layer's weights into shared
 * memory.  Nothing is in flight for the missing piece; the warps that wait for it run into the
 * wait limit, the kernel returns, `out` holds unspecified values and dhq_last_status reports
 * DHQ_ERR_TIMEOUT.  Later launches are normal.  Set a short limit first (dhq_set_wait_limit).
 * UNSUPPORTED for a handle without a fused kernel (one that runs layer by layer).
 */
DHQ_API dhq_status_t dhq_debug_stall_next_forward(dhq_handle_t h);

/*
 * Read back one prepared layer (1-based).  Synchronizes the handle's preparation work.
 *   codes       host [M][K] int8, row-major, unswizzled (M, K as in dhq_debug_bufs_t), or NULL.
 *   w_scales    host [M] fp32 (per-tensor: the same value M times), or NULL.
 *   act_absmax  host, one fp32: the frozen per-tensor a_l, or NaN if not frozen / per token;
 *               or NULL.
 * Errors: INVALID_ARG (layer out of range), CUDA.
 */
DHQ_API dhq_status_t dhq_get_layer(dhq_handle_t h, int layer, int8_t *codes, float *w_scales,
                                   float *act_absmax);

/*
 * Forward pass for callers that must not allocate device memory.  (The paper has no
 * counterpart; this is a deployment variant of dhq_forward_debug without the dumps.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a framework that owns
 * the whole device heap through its own caching allocator, in a process whose memory budget is
 * fixed at start-up, or in a latency-critical loop where an allocation's implicit device
 * synchronisation is not acceptable.  The other layer-by-layer entry points grow scratch
 * buffers with cudaMalloc on demand; this one never does.  It runs the same per-layer kernel,
 * but the activations that travel between layers live in a fixed array that is part of the
 * library image itself: 2 x DHQ_STATIC_MAX_TOKENS x 512 floats = 16 MiB, which every GPU that
 * loads the library carries until the process exits, whether or not this call is ever used.
 *
 *   coords  device [n][2] fp32, out device [n][d_L] fp32, as for dhq_forward.
 *   n       0 .. DHQ_STATIC_MAX_TOKENS; a larger n returns DHQ_ERR_TOO_LARGE and enqueues
 *           nothing (split the batch and call again once the previous call has finished).
 * Results equal dhq_forward's bit for bit.  Per-tensor activation scales must already be frozen
 * (dhq_calibrate, which does allocate, or an earlier dhq_forward): otherwise NOT_CALIBRATED.
 * The call makes no cudaMalloc/cudaFree and calls no allocating library routine.
 *
 * Set-up: the first call on each device looks up the device address of the scratch array
 * (once per device, with that device current) and keeps it; make that first call before any
 * stream capture begins.
 * Sharing: all handles and all calls on a device use the same array, and it keeps whatever the
 * last call left there.  Nothing in it needs clearing, because each layer pass writes every
 * value that the next pass reads; but two calls whose kernels overlap on the GPU (different
 * streams, no ordering between them) race on it and both give wrong results.  Order them.
 */
#define DHQ_STATIC_MAX_TOKENS 4096
DHQ_API dhq_status_t dhq_forward_static_scratch(dhq_handle_t h, const float *coords, int64_t n,
                                                float *out, void *stream);

/*
 * A prepared (and, if it was, calibrated) handle as a block of host memory, and back: so that the
 * weight-side work of Eq. 4-5 and the calibration run once and every GPU or process that serves
 * the same network (coordinates are independent, Section II-A, so the work splits over GPUs by
 * coordinate blocks) starts from the same bytes.
 *   dhq_export  host_buf NULL: only *needed is written (size query).  Otherwise capacity must be
 *               >= *needed (TOO_LARGE if not); synchronizes the device and fills host_buf.
 *   dhq_import  builds a new handle on the current device from such a block; the block is
 *               checked (magic, version, sizes against the configuration it states, checksum of
 *               the arrays): INVALID_ARG if anything is off.  The caller may release host_buf when
 *               the call returns.  Results of the new handle equal the exported one's bit for bit.
 * The block is the library's own format, valid for this library version and sm_100a layouts.
 * Errors: INVALID_ARG, UNSUPPORTED, TOO_LARGE, ALLOC, CUDA.
 */
DHQ_API dhq_status_t dhq_export(dhq_handle_t h, void *host_buf, int64_t capacity, int64_t *needed);
DHQ_API dhq_status_t dhq_import(const void *host_buf, int64_t bytes, void *stream, dhq_handle_t *out);

/* Layer sizes as the library pads them: K, M of layer `layer` (1-based).  Either may be NULL. */
DHQ_API dhq_status_t dhq_layer_dims(dhq_handle_t h, int layer, int *K, int *M);

/*
 * Device-side status of the handle: DHQ_OK, or DHQ_ERR_TIMEOUT if a bounded wait inside a
 * kernel ran out since the last call.  Synchronizes the device and clears the word.
 */
DHQ_API dhq_status_t dhq_last_status(dhq_handle_t h);

/*
 * The SM clock that the handle's last dhq_forward_fused_debug launch really ran at: in that
 * instantiation of the fused kernel two threads of the first CTA read the SM's cycle counter and
 * the global nanosecond timer before and after the work; sm_mhz = cycles / time.  (NVML reports the
 * clock the driver asks for; inside the launches the SMs were seen 4-8 % below it.  The timed
 * instantiations do not carry the probe: a dhq_forward_fused_debug call without dump buffers does
 * the same work at nearly the same speed and serves as the clock measurement.)  milliseconds: that
 * CTA's run time, close to the launch's.  Synchronizes the device.  Either pointer may be NULL.
 * (No counterpart in the paper: measurement.)
 * Errors: INVALID_ARG (no such launch yet), UNSUPPORTED (handle runs layer by layer), CUDA.
 */
DHQ_API dhq_status_t dhq_last_launch_clock(dhq_handle_t h, double *sm_mhz, double *milliseconds);

/* Number of kernels the library has launched for this handle since it was created. */
DHQ_API int64_t dhq_launch_count(dhq_handle_t h);

/* Waits for the handle's outstanding work, then frees everything it owns.  NULL is ignored. */
DHQ_API void dhq_destroy(dhq_handle_t h);

DHQ_API const char *dhq_status_string(dhq_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* DHQ_H_ */
