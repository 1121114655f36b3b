/*
 * wfq.h - C ABI of the group-wise int8-quantized Winograd convolution F(m,3) for
 * NVIDIA B200 (sm_100a).
 *
 * The library evaluates y = conv2d(x, w, stride 1, padding 1, no bias) (deep-learning
 * cross-correlation) for 3x3 filters through the quantized Winograd pipeline of the
 * paper "Data-Free Group-Wise Fully Quantized Winograd Convolution via Learnable
 * Scales" (Section 3.1 for the algorithm, Section 4.1 for the scaled transforms and
 * the quantized Hadamard stage, Eq. quant-Y):
 *
 *   W = S_G V_G w V_G^T S_G        filter transform, offline        (wfq_prepare_filters)
 *   X = S_B V_B x V_B^T S_B        input transform, fp32
 *   Xq, sX = Q(X)                  int8 codes + one fp32 scale per group of
 *                                  `group_size` consecutive input channels, per
 *                                  Winograd position and tile (dynamic abs-max)
 *   acc[g] = sum_{c in g} Xq Wq    int8 x int8 -> int32 on the tensor cores,
 *                                  one matrix product per Winograd position
 *   Y = sum_g acc[g] sX[g] sW[g]   per-group dequantization into fp32
 *   y = V_A S_A Y S_A V_A^T        output transform, fp32, cropped to H x W
 *
 * Notation: n = m + 2, P = n*n positions (p = i*n + j), TH = ceil(H/m),
 * TW = ceil(W/m), T = N*TH*TW tiles (t = (img*TH + th)*TW + tw), G = C/group_size.
 *
 * Quantizer (per group, fp32): amax = max|v|; if amax < 1e-30 the scale is 0 and all
 * codes are 0; otherwise scale = amax/127, inv = 127/amax (both correctly rounded) and
 * code = clamp(round_half_even(v*inv), -127, 127).
 *
 * General rules
 *   - All functions return a wfq_status_t; nothing throws, aborts or traps.
 *   - Arguments are validated before any device work is launched.
 *   - "device" pointers are CUDA device pointers of the current device, "host"
 *     pointers are ordinary host memory.  `stream` is a cudaStream_t passed as void*
 *     (NULL = the default stream).
 *   - Work is asynchronous on `stream` unless stated; buffers must stay valid until
 *     that work has completed.  One plan must not be used from two threads or two
 *     streams at the same time (its workspace is shared).
 *   - The library needs a device of compute capability 10.x; on anything else the
 *     launching calls return WFQ_ERR_UNSUPPORTED or WFQ_ERR_CUDA.  There is no CPU
 *     fallback.
 */
#ifndef WFQ_H_
#define WFQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct wfq_plan wfq_plan_t; /* opaque, owned by the library */

typedef enum {
    WFQ_OK = 0,
    WFQ_ERR_INVALID_ARG = 1,  /* NULL pointer, non-positive size, bad enum value */
    WFQ_ERR_UNSUPPORTED = 2,  /* valid request outside the supported set */
    WFQ_ERR_ALLOC = 3,        /* host or device allocation failed */
    WFQ_ERR_NOT_PREPARED = 4, /* workspace or filters missing */
    WFQ_ERR_CUDA = 5,         /* a CUDA runtime/driver call failed */
    WFQ_ERR_TIMEOUT = 6,      /* a bounded device-side wait expired (status word) */
    WFQ_ERR_SCRATCH_TOO_SMALL = 7 /* problem larger than the library's built-in scratch */
} wfq_status_t;

typedef enum { WFQ_F32 = 0, WFQ_F16 = 1, WFQ_BF16 = 2 /* output only */ } wfq_dtype_t;

/* Memory layout of the input x: [N][C][H][W] (default) or [N][H][W][C]. */
typedef enum { WFQ_NCHW = 0, WFQ_NHWC = 1 } wfq_layout_t;

/* Activation applied by the output transform after the optional bias. */
typedef enum { WFQ_ACT_NONE = 0, WFQ_ACT_RELU = 1, WFQ_ACT_SILU = 2 } wfq_activation_t;

/* Buffers that wfq_debug_get can expose (all device memory). */
typedef enum {
    WFQ_BUF_XQ = 0,     /* int8  Xq[P][T][C]            (workspace)  */
    WFQ_BUF_SX = 1,     /* fp32  sX[P][G][Ts], Ts = T rounded up to 128; entries t >= T
                           are not written (workspace)  */
    WFQ_BUF_WQ = 2,     /* int8  Wq[P][K][C]            (plan-owned) */
    WFQ_BUF_SW = 3,     /* fp32  sW[P][G][Kp], Kp = K rounded up to 128, zero for k >= K
                           (plan-owned) */
    WFQ_BUF_Y = 4,      /* fp32  Y[P][K][Tp], Tp = T rounded up to 32 (workspace) */
    WFQ_BUF_STATUS = 5  /* int32 status[4]: {code, where, block, aux} (plan-owned) */
} wfq_buffer_t;

/* Test and profiling switches of wfq_plan_set_debug_option. */
typedef enum {
    WFQ_DEBUG_WAIT_CYCLES = 0,      /* limit of every device-side wait in SM clock cycles
                                       (default 2e9, about a second; at least 1000) */
    WFQ_DEBUG_SKIP_INPUT_ITEM = 1,  /* work item whose input strip the tensor-core input
                                       transform's producer does not load (-1 = none): the
                                       waits for it run out, the kernel records
                                       WFQ_ERR_TIMEOUT in the status word and ends by itself */
    WFQ_DEBUG_INPUT_TRANSFORM_KERNEL = 2, /* 0: the library chooses; 1: the cp.async kernel;
                                       2: the tensor-core kernel wherever it applies (fp16 input,
                                       groups of 32 or 64, C a multiple of 64, 16-byte aligned x,
                                       a shape its TMA or bulk staging can describe) */
    WFQ_DEBUG_SKIP_GEMM_STAGE = 3,  /* operand stage (counted from 0) whose loads the first
                                       CTA of the contraction kernel does not issue (-1 =
                                       none); same purpose as WFQ_DEBUG_SKIP_INPUT_ITEM */
    WFQ_DEBUG_GEMM_SHAPE = 4        /* 0: the library chooses the contraction's orientation and
                                       column block; else 100 * orientation (1: accumulator rows are
                                       tiles, 2: rows are output channels) + columns per unit (16 or
                                       64 for orientation 1; 16, 32, 48 or 64 for orientation 2).
                                       Results do not depend on it; for timing experiments */
} wfq_debug_option_t;

/*
 * Create a plan for one layer: x[N][C][H][W] -> y[N][K][H][W] evaluated as F(m,3)
 * (Section 3.1: output tile m x m, filter r x r, input tile (m+r-1)^2).
 * Supported: r = 3; m in {2, 4, 6} (F(4,3) and F(6,3) are the paper's tiles; F(2,3) is the textbook
 * tile with the matrices B^T = [1 0 -1 0; 0 1 1 0; 0 -1 1 0; 0 1 0 -1], G = [1 0 0; 1/2 1/2 1/2;
 * 1/2 -1/2 1/2; 0 0 1], A^T = [1 1 1 0; 0 1 -1 -1] as its standard scaling); bits = 8; group_size a multiple of 32, at most 256,
 * dividing C; N, C, K, H, W >= 1; P*T*C, P*K*C and N*K*H*W below 2^31.
 * Returns WFQ_ERR_INVALID_ARG for NULL/non-positive arguments and
 * WFQ_ERR_UNSUPPORTED for anything else outside this set.  Synchronous, host-only
 * (no device is touched).
 */
wfq_status_t wfq_plan_create(wfq_plan_t **out, int N, int C, int K, int H, int W, int m,
                             int r, int group_size, int bits);

/* Element type of x in wfq_conv_forward (default WFQ_F32).  Call before forward. */
wfq_status_t wfq_plan_set_input_dtype(wfq_plan_t *plan, wfq_dtype_t dtype);

/*
 * Optional epilogue fused into the output transform (the paper's layers are followed by a
 * bias and an activation; the paper itself gives no formula for them, Section 3.1 defines
 * the convolution only): y = act(conv(x, w) + bias[k]).
 *   bias_dev  device, fp32 [K], caller-owned and kept alive while the plan is used; NULL = none
 *   act       WFQ_ACT_NONE, WFQ_ACT_RELU (max(t, 0)) or WFQ_ACT_SILU (t / (1 + exp(-t)))
 * Host only; takes effect from the next forward call.  Default: no bias, no activation.
 */
wfq_status_t wfq_plan_set_epilogue(wfq_plan_t *plan, const float *bias_dev, wfq_activation_t act);

/*
 * Layout of x.  With WFQ_NHWC, `x_dev` / `x_host` of the forward calls hold x[N][H][W][C] (same
 * element type as set by wfq_plan_set_input_dtype) and x_dev must be 16-byte aligned
 * (WFQ_ERR_CUDA from the forward call otherwise); the input transform then stages each work
 * item's strip with one TMA tensor copy (channels innermost) instead of per-thread copies.  The
 * result is the same bit for bit as for the NCHW tensor with the same values; y stays
 * [N][K][H][W].  Not available together with the integer input transform.  Host only.
 */
wfq_status_t wfq_plan_set_input_layout(wfq_plan_t *plan, wfq_layout_t layout);

/*
 * Element type of the output y: WFQ_F32 (default), WFQ_F16 or WFQ_BF16.  With a 16-bit type the
 * output transform rounds each result once (to nearest even, after bias and activation) and
 * `y_nkhw_dev` / `y_host` of the forward calls point at 2-byte storage of the same [N][K][H][W]
 * shape (the parameters keep their `float *` type; alignment requirements are unchanged).
 * Host only.
 */
wfq_status_t wfq_plan_set_output_dtype(wfq_plan_t *plan, wfq_dtype_t dtype);

/*
 * Bit width of the filter codes: 8 (default) or 4 (WFQ_ERR_UNSUPPORTED otherwise).  With 4 the
 * offline filter path quantizes each channel group of the transformed filters to codes in
 * [-7, 7] with scale = amax / 7 (the quantizer of the header comment with 7 in place of 127): the
 * "W4A8" setting of the paper's experiments (Section 5), which the paper applies to its other
 * layers and which is offered here for the Winograd layers as well.  Activations stay at 8 bits.
 * On the device the codes remain one per byte, because the contraction is an int8 tensor-core
 * product either way and is not bound by the filter stream; the exported blob stores two per
 * byte.  Changing the width invalidates prepared filters: call wfq_prepare_filters (or
 * wfq_filters_import) afterwards.  Host only.
 */
wfq_status_t wfq_plan_set_weight_bits(wfq_plan_t *plan, int bits);

/*
 * The paper's fully quantized transforms (Section 4.1), off by default.
 *   quant_input  1: the input transform runs on integer codes (Eq. quant-B): x is quantized to 8
 *                bits with one scale per (tile, channel group) over the group's n x n patches,
 *                S_B V_B to 8 bits with one scale, the two matrix products are integer products
 *                and the result times s_qB^2 s_qx is what the group quantizer of the contraction
 *                sees.  0: floating-point input transform.
 *   y_mode       WFQ_Y_FP32: floating-point output transform; WFQ_Y_TILE / WFQ_Y_ROW: the output
 *                transform runs on integer codes (Eq. quant-y) with V_A S_A quantized to 8 bits
 *                with one scale and Y with one scale per (tile, output channel), or with one
 *                scale per row of the n x n matrix and, after the first product, one per column
 *                (Section 3.2: Y needs a scale per tile or per row / column).
 * With an integer output transform the scale vectors given to wfq_prepare_filters change the
 * result (this is where the paper's learned scales act); with the floating-point transforms they
 * are numerically neutral.  Group sizes: multiples of 32 up to 256.  Host only; takes effect from
 * the next forward call.  These kernels are reference-speed implementations.
 */
typedef enum { WFQ_Y_FP32 = 0, WFQ_Y_TILE = 1, WFQ_Y_ROW = 2 } wfq_y_quant_t;
wfq_status_t wfq_plan_set_full_quant(wfq_plan_t *plan, int quant_input, wfq_y_quant_t y_mode);

/*
 * Bytes of caller-owned device scratch the plan needs (Xq + sX + Y, each region
 * 1024-byte aligned).  Returns 0 for a NULL plan.
 */
size_t wfq_plan_workspace_bytes(const wfq_plan_t *plan);

/*
 * Hand the plan its scratch memory: `dev_ptr` device memory, 1024-byte aligned, at
 * least wfq_plan_workspace_bytes() long, owned by the caller and kept alive while the
 * plan is used.  Builds the TMA descriptor of Xq.  WFQ_ERR_INVALID_ARG if too small or
 * misaligned.
 */
wfq_status_t wfq_plan_set_workspace(wfq_plan_t *plan, void *dev_ptr, size_t bytes);

/*
 * Offline filter path (Section 4.1, W = S_G V_G w V_G^T S_G; "weight transformation can
 * be done offline with high precision"): transform in fp64, round once to fp32,
 * quantize every group of `group_size` consecutive input channels per (position,
 * output channel), and store the codes position-major (the paper's offline reordering
 * of weights to compute order).
 *   w_dev    device, fp32 [K][C][3][3]
 *   sB_host  host, n floats, diagonal of S_B (NULL = standard scales of the paper)
 *   sG_host  host, n floats, diagonal of S_G (NULL = standard scales)
 *   sA_host  host, n floats, diagonal of S_A (NULL = 1/(sB*sG), Eq. scaling_condition,
 *            evaluated in fp64 and rounded to fp32)
 * All scales must be finite and nonzero (signs are allowed).  The first call on a plan
 * allocates the plan-owned Wq/sW buffers and the status word with cudaMalloc (which may
 * synchronise the device); every call takes the fp32 temporary between its two kernels
 * from the stream-ordered allocator (cudaMallocAsync / cudaFreeAsync on `stream`), so
 * later calls neither block nor synchronise.  Asynchronous on `stream`; may be called
 * again to replace the filters.  The first library call that meets a device (this one or
 * wfq_plan_set_workspace) also sets that device's kernel attributes; make it outside any
 * stream capture.
 */
wfq_status_t wfq_prepare_filters(wfq_plan_t *plan, const float *w_dev, const float *sB_host,
                                 const float *sG_host, const float *sA_host, void *stream);

/*
 * Filter quantization for callers that must not allocate.  (The paper has no
 * counterpart to this call; it exists for integration reasons only.)
 *
 * wfq_prepare_filters obtains its buffers with cudaMalloc.  Some hosts of this library
 * cannot do that at the point where filters arrive: code running inside a framework
 * whose memory pool owns the whole device, a real-time loop where the allocator's
 * implicit device synchronisation is not acceptable, or a process whose device memory
 * was fully budgeted at start-up.  This call produces the same codes and scales as
 * wfq_prepare_filters (same kernels, same arithmetic) and allocates nothing: no
 * cudaMalloc/cudaFree, no host allocation, no library routine that allocates.  The fp32
 * transformed filters it needs between its two kernels are kept in one array that is
 * part of the library's device image, WFQ_STATIC_SCRATCH_FLOATS floats (16 MiB); every
 * GPU on which the library is loaded holds that array until the process exits.
 *
 *   w_dev        device, fp32 [K][C][3][3]                               (input)
 *   sG_host      host, m+2 floats, diagonal of S_G; NULL = standard scales
 *   wq_dev       device, int8 [P][K][C], caller-owned                    (output)
 *   sw_dev       device, fp32 [P][C/group_size][K], caller-owned         (output)
 *   m in {2,4,6}; group_size a multiple of 32, at most 256, dividing C.
 *
 * Limit: (m+2)^2 * K * C <= WFQ_STATIC_SCRATCH_FLOATS, otherwise
 * WFQ_ERR_SCRATCH_TOO_SMALL is returned and nothing is launched.  Other argument errors
 * are reported as in wfq_prepare_filters.  Asynchronous on `stream`.
 *
 * The first call on each device looks up the device address of the built-in array
 * (with that device current); make that first call outside any stream capture.  All
 * calls on a device share the one array: it still holds the previous call's values
 * when a call starts (harmless, every element that is read is written first by the
 * same call, so nothing needs clearing), and two calls whose kernels can overlap on
 * the GPU (different streams, or different host threads) race on it.  Serialise them.
 * The looked-up address is cached per device ordinal for the life of the process;
 * cudaDeviceReset invalidates it, so do not call this function after a device reset.
 */
#define WFQ_STATIC_SCRATCH_FLOATS (4u * 1024u * 1024u)
wfq_status_t wfq_quantize_filters_static(const float *w_dev, int K, int C, int m, int group_size,
                                         const float *sG_host, int8_t *wq_dev, float *sw_dev,
                                         void *stream);

/*
 * The hot path: input transform + group quantization, per-position int8 tensor-core
 * contraction with per-group dequantization, output transform.
 *   x_dev  device, [N][C][H][W] in the plan's input dtype, 4-byte aligned
 *   y_dev  device, fp32 [N][K][H][W], 16-byte aligned
 * Three kernels are enqueued on `stream`; no host synchronisation and no other runtime
 * call, except that a TMA descriptor of x is re-encoded (host only) when x_dev differs
 * from the previous call's.  Requires a workspace and prepared filters
 * (WFQ_ERR_NOT_PREPARED otherwise).
 */
wfq_status_t wfq_conv_forward(wfq_plan_t *plan, const void *x_dev, float *y_dev, void *stream);

/*
 * Prepared filters as a host blob, so that wfq_prepare_filters can run once, offline, and a later
 * process only loads its result (the filter path is offline in the paper as well, Section 4.1).
 * The blob holds a 256-byte header (layer shape, tile and group size, the three scale vectors in
 * fp64, the weight bit width), Wq [P][K][C] and sW [P][G][Kp] fp32; it is tied to those parameters,
 * not to the batch size or the image size.  Wq is one int8 code per byte for 8-bit weights and two
 * codes per byte for 4-bit weights (byte j: code 2j in the low nibble, code 2j+1 in the high nibble,
 * two's complement), which halves the blob.
 *   wfq_filters_bytes   size of the blob for this plan
 *   wfq_filters_export  host_buf (host, >= that size, caller-owned) receives the blob of a
 *                       prepared plan; synchronous with respect to `stream`
 *   wfq_filters_import  makes the plan prepared from a blob written for the same C, K, tile and
 *                       group size (WFQ_ERR_INVALID_ARG otherwise, plan unchanged); the plan takes
 *                       the blob's weight bit width; the blob is copied before the call returns;
 *                       a CUDA error during the copy (WFQ_ERR_CUDA) leaves the plan unprepared
 */
size_t wfq_filters_bytes(const wfq_plan_t *plan);
wfq_status_t wfq_filters_export(wfq_plan_t *plan, void *host_buf, size_t bytes, void *stream);
wfq_status_t wfq_filters_import(wfq_plan_t *plan, const void *host_buf, size_t bytes, void *stream);

/*
 * Same computation with HOST buffers: copies x to the device, runs the three kernels,
 * copies y back, then waits for `stream` (synchronous).  The plan allocates device
 * staging for x and y on first use.  x_host/y_host should be pinned for full copy speed.
 * Batches of three or more images with more than 12 MB to move are cut into chunks of
 * whole images that alternate between two streams owned by the plan (created on first
 * use, ordered after the work already on `stream`, and `stream` waits for them), so that
 * copies in, kernels and copies out overlap; the results are identical to the unchunked
 * path.
 */
wfq_status_t wfq_conv_forward_host(wfq_plan_t *plan, const void *x_host, float *y_host,
                                   void *stream);

/*
 * The same without the final wait: the copies and kernels are enqueued and the call returns;
 * y_host holds the result once `stream` has been waited for (all internal work is joined to
 * `stream`).  x_host and y_host must stay valid, and x_host unmodified, until then; pageable
 * host memory makes the copies synchronous with respect to the host.  The plan's staging
 * buffers are reused by the next call on the same plan, which is ordered after this one when it
 * uses the same stream; calls on different plans may use different streams so that the copy in
 * of one layer overlaps the copy out of another.
 */
wfq_status_t wfq_conv_forward_host_async(wfq_plan_t *plan, const void *x_host, float *y_host,
                                         void *stream);

/* The three stages of wfq_conv_forward, separately (tests and profiling). */
/* Stage 1 (X = S_B V_B x V_B^T S_B, then Q): x_dev -> workspace Xq, sX. */
wfq_status_t wfq_input_transform_quantize(wfq_plan_t *plan, const void *x_dev, void *stream);
/* Stage 2 (Eq. quant-Y): workspace Xq, sX and the plan's Wq, sW -> workspace Y. */
wfq_status_t wfq_gemm_dequantize(wfq_plan_t *plan, void *stream);
/* Stage 3 (y = V_A S_A Y S_A V_A^T): workspace Y -> y_dev. */
wfq_status_t wfq_output_transform(wfq_plan_t *plan, float *y_dev, void *stream);

/*
 * Raw int32 group accumulators of stage 2, before any scaling:
 *   acc_dev[p][t][k][g] = sum_{c in group g} Xq[p][t][c] * Wq[p][k][c]
 * computed by the same tensor-core kernel as wfq_gemm_dequantize from the operands
 * currently in the workspace (Xq) and the plan (Wq).  acc_dev: device, int32,
 * P*T*K*G elements.
 */
wfq_status_t wfq_debug_gemm_acc32(wfq_plan_t *plan, int32_t *acc_dev, void *stream);

/*
 * Measurement aid: the rate of the int8 tensor pipe as this library drives it.  Enqueues on
 * `stream` one CTA per SM, each issuing `mmas_per_sm` (a multiple of 4) accumulating
 * tcgen05.mma kind::i8 instructions of shape 128 x n_cols x 32 (n_cols in {64, 128, 256}) on
 * operands resident in shared memory, and stores in *ops (host) the number of integer
 * operations (2 per multiply-add) the launch performs; the caller times the launch.  No
 * global memory is read or written.  Needs prepared filters (for the status word).
 */
wfq_status_t wfq_debug_int8_mma_rate(wfq_plan_t *plan, int n_cols, int mmas_per_sm, long long *ops,
                                     void *stream);

/*
 * Set a test/profiling switch of the plan (see wfq_debug_option_t).  Host only.
 * WFQ_ERR_INVALID_ARG for an unknown option or a value outside its range.
 */
wfq_status_t wfq_plan_set_debug_option(wfq_plan_t *plan, wfq_debug_option_t option, long long value);

/*
 * Device address and size of an internal buffer (see wfq_buffer_t for layouts).
 * Tests read intermediates from these and may overwrite the workspace ones to feed a
 * later stage with chosen operands.
 */
wfq_status_t wfq_debug_get(wfq_plan_t *plan, wfq_buffer_t which, void **dev_ptr, size_t *bytes);

/*
 * Read (synchronously, after waiting for `stream`) the device status word that the
 * kernels set when one of their bounded waits expires.  Returns WFQ_OK or
 * WFQ_ERR_TIMEOUT; `where` (may be NULL) receives an identifier of the wait.
 */
wfq_status_t wfq_check_device_status(wfq_plan_t *plan, void *stream, int *where);

/* Release the plan and everything it owns (not the workspace).  NULL is accepted. */
wfq_status_t wfq_plan_destroy(wfq_plan_t *plan);

/* Static string for a status code. */
const char *wfq_status_string(wfq_status_t status);

/* Library version as major*100 + minor. */
int wfq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* WFQ_H_ */
