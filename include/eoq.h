/*
 * eoq.h -- C ABI of the EOQ 8-bit integer training layer on NVIDIA sm_100a.
 *
 * The library implements the quantized convolution layer of the BN-free Fixup
 * residual network of "Towards Efficient Full 8-bit Integer DNN Online Training
 * on Resource-limited Devices without Batch Normalization" (arXiv 2105.13890):
 * forward, error back-propagation and weight gradient, each an int8 x int8 ->
 * int32 implicit GEMM, fused with the paper's quantizers, plus the 8-bit update.
 *
 * Conventions for every entry point
 *   - A quantized tensor is (integer codes, exponent p): real value = code * 2^p.
 *     Forward-side tensors (activations, weights, gamma, biases) sit on the grid
 *     of Q(., 8), p = -7, and carry no exponent.  Outputs of the scale quantizer
 *     SQ carry one int32 exponent per tensor, kept in DEVICE memory so that no
 *     host round trip separates producer and consumer.
 *   - All bit widths are 8 (Sec. 5.1).  R(.) rounds to nearest, ties to even.
 *   - Layouts: activations and errors NHWC int8; weights [c_out][kh][kw][c_in]
 *     int8.  c_in and c_out must be multiples of 16 (pad with zero channels); c_in may
 *     also be 8 for a first layer that takes the filter-row path (eoq_conv_desc_t).
 *   - Pointers named in a "device" list are device pointers the caller owns; the
 *     library never allocates or frees tensor memory.  Tensor pointers must be
 *     16-byte aligned.  Scratch memory is the caller's `workspace` (device, 256-byte
 *     aligned, at least eoq_workspace_size() bytes; contents are undefined on
 *     entry and on return).  The handle owns only a few hundred bytes of device
 *     state (status word, small reduction cells) and a few internal streams and
 *     events.  A handle serves one call at a time: calls that may overlap on the
 *     device (different streams) need a handle and a workspace each.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls enqueue work and return without synchronising, except
 *     eoq_create, eoq_destroy and eoq_last_status.  A call may issue independent
 *     parts of its work on the handle's internal streams, forked from and joined
 *     back into `stream` with events (under stream capture these become graph
 *     edges); when the call returns, everything it enqueued is ordered before
 *     whatever is enqueued on `stream` next.
 *   - Every function returns an eoq_status_t.  Nothing throws, traps or aborts.
 *     Conditions only the device can see (a wait that ran out, a non-finite
 *     input, an all-zero SQ input) are OR-ed into the handle's device status
 *     word; eoq_last_status() reads and clears it.
 */
#ifndef EOQ_H
#define EOQ_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define EOQ_API __attribute__((visibility("default")))
#else
#define EOQ_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct eoq_handle_s *eoq_handle_t;

typedef enum {
    EOQ_OK = 0,
    EOQ_ERR_BAD_ARG = 1,     /* null pointer, non-positive size, inconsistent geometry */
    EOQ_ERR_ALIGNMENT = 2,   /* pointer not 16-byte aligned, channel count not a multiple of 16 (or c_in = 8) */
    EOQ_ERR_UNSUPPORTED = 3, /* geometry outside what the kernels cover */
    EOQ_ERR_WORKSPACE = 4,   /* workspace missing, misaligned or too small */
    EOQ_ERR_RANGE = 5,       /* a scalar code outside its range */
    EOQ_ERR_CUDA = 6         /* a CUDA call failed; see eoq_last_cuda_error() */
} eoq_status_t;

/* Bits of the device status word returned by eoq_last_status(). */
#define EOQ_DEV_TIMEOUT 1u   /* a bounded wait inside a kernel ran out; results of that call are invalid */
#define EOQ_DEV_NONFINITE 2u /* eoq_quantize met a NaN or an infinity */
#define EOQ_DEV_SQ_ZERO 4u   /* a scale quantizer saw an all-zero tensor (codes 0, exponent passed through) */
#define EOQ_DEV_RANGE 8u     /* an input exponent outside the supported range */

typedef enum { EOQ_Q = 0, EOQ_CQ = 1, EOQ_SQ = 2 } eoq_qmode_t;
typedef enum { EOQ_ROUND_RNE = 0, EOQ_ROUND_STOCHASTIC = 1 } eoq_round_t;
typedef enum { EOQ_PASS_FWD = 0, EOQ_PASS_DGRAD = 1, EOQ_PASS_WGRAD = 2 } eoq_pass_t;

/* Geometry of one convolution: input [n,h,w,c_in], filter kh x kw, square stride and padding.
 * Output spatial size is (h + 2 pad - kh) / stride + 1 by (w + 2 pad - kw) / stride + 1.
 * x_wmargin (normally 0): the INPUT tensor x is stored with that many zero pixels before and after every image
 * row, i.e. as [n][h][w + 2 x_wmargin][c_in] with the image in the middle (eoq_quantize_image writes this form).
 * The margins are part of the zero padding, not of the image.  With c_in = 16 or 8, a filter 5 to 8 taps wide and
 * a margin of at least max(pad, (wo-1) stride - pad + 8 - w) pixels (4 for the 7x7 stride-2 first layer of the
 * ImageNet ResNets) a whole filter row is fetched as one 128- or 64-byte run (the filter-row path), which is
 * several times faster than one 16-byte fetch per tap.  c_in = 8 (an RGB image padded to 8 channels) halves the
 * padded reduction length again; it exists only on this path and needs an even stride, an even w and an even
 * x_wmargin - pad (5 for that first layer), else forward and wgrad return EOQ_ERR_UNSUPPORTED; dgrad does not
 * take c_in = 8 (the network input receives no error).  Outputs and the error tensors never carry margins. */
typedef struct {
    int n, h, w, c_in, c_out, kh, kw, stride, pad, x_wmargin;
} eoq_conv_desc_t;

/* Creates a handle on CUDA device `device` (makes it current).  Synchronises. */
EOQ_API int eoq_create(eoq_handle_t *handle, int device);
EOQ_API int eoq_destroy(eoq_handle_t handle);

/* Bytes of workspace a pass needs for this geometry (a multiple of 256; may be 0). */
EOQ_API int eoq_workspace_size(const eoq_conv_desc_t *desc, int pass, size_t *bytes);

/*
 * Forward chain of one layer (Sec. 3.2.1, first equation block):
 *   x1 = x0 + Q_b(b1)         (zero halo: padding applies to x1)
 *   x2 = Q_a1(conv(x1, Q_w(w)))  code = sat16(R(acc / 2^s)), s = -x_exp (7 when x_exp is NULL)
 *   x3 = Q_gamma(gamma) * x2
 *   x4 = x3 + Q_b(b2) [+ shortcut]
 *   x5 = Q_a2(relu(x4))       code = sat(R(max(x4,0) / 2^7), -127, 127);  relu = 0 keeps x4's sign
 * device in : x [n,h,w,c_in] int8; x_exp (int32, exponent of x; NULL means -7); w; shortcut
 *             [n,ho,wo,c_out] int8 at p = -7 or NULL.
 * host in   : b1_c, gamma_c, b2_c integer codes at p = -7 (gamma = 1 is 128), each within int16.
 * device out: x5 [n,ho,wo,c_out] int8; optional x2 (int16, same shape), relu_mask (bit i of the
 *             NHWC-linear element index i in byte i/8, bit i%8: [x4 > 0]) and acc_dump (int32 conv
 *             accumulators including the b1 term) -- each may be NULL.
 * Errors: BAD_ARG, ALIGNMENT, UNSUPPORTED (kh*kw > 64 taps), RANGE, WORKSPACE, CUDA.
 */
EOQ_API int eoq_conv_fwd(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *x, const int32_t *x_exp,
                 int32_t b1_c, const int8_t *w, int32_t gamma_c, int32_t b2_c, const int8_t *shortcut, int relu,
                 int8_t *x5, int16_t *x2, uint8_t *relu_mask, int32_t *acc_dump, void *workspace,
                 size_t workspace_bytes, void *stream);

/*
 * The same forward chain for a training loop whose scalars live in device memory and whose weights change only in
 * the update (Sec. 3.2.1, first equation block; Sec. 3.2.3 for what changes them).
 *   scalars (device, three int32: b1_c, gamma_c, b2_c, codes at p = -7) replace the three host arguments: a step
 *   recorded once into a CUDA graph then reads the current codes at every replay.  Codes outside 16 bits, or a b1
 *   that would let the accumulator leave int32, raise EOQ_DEV_RANGE and are clamped.
 *   w_prep (device, 256-byte aligned, eoq_weight_prep_size() bytes) holds what eoq_weight_prep derived from w: the
 *   per-border-class weight sums of the b1 term and, on the filter-row path, the row-padded weights.  With w_prep
 *   no helper kernel runs in front of the convolution.  w_prep = NULL states that the layer has no bias before its
 *   convolution: scalars[0] must then be 0 (anything else raises EOQ_DEV_RANGE and counts as 0); the filter-row
 *   path always needs w_prep.
 * Everything else is as in eoq_conv_fwd; there is no accumulator dump and no workspace.
 */
EOQ_API int eoq_conv_fwd_dev(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *x, const int32_t *x_exp,
                     const int32_t *scalars, const int8_t *w, const void *w_prep, const int8_t *shortcut, int relu,
                     int8_t *x5, int16_t *x2, uint8_t *relu_mask, void *stream);

/*
 * What the forward pass needs from the weights besides the codes themselves (x1 = x0 + Q_b(b1) with a zero halo,
 * Sec. 3.2.1: conv(x1) = conv(x0) + b1 * sum of the weights of the taps inside the image).  It depends on w and the
 * geometry only, so it is formed once per weight version -- after initialisation and after every eoq_update --
 * for `num` layers in one launch per 32 layers.
 * host in   : descs[num]; arrays (host memory) of device pointers w[i] and prep[i] (256-byte aligned,
 *             eoq_weight_prep_size(&descs[i]) bytes each).
 */
EOQ_API int eoq_weight_prep_size(const eoq_conv_desc_t *desc, size_t *bytes);
EOQ_API int eoq_weight_prep(eoq_handle_t handle, int num, const eoq_conv_desc_t *descs, const int8_t *const *w,
                    void *const *prep, void *stream);

/*
 * Error back-propagation through the convolution (Sec. 3.2.1, second equation block):
 *   e4 = Q_e(e3 * Q_w(w)), the transposed convolution followed by SQ over the whole tensor.
 * device in : e3 [n,ho,wo,c_out] int8 with exponent *e3_exp; w.
 * device out: e4 [n,h,w,c_in] int8; *e4_exp = *e3_exp - 7 + t - 7 with 2^t the scale of SQ;
 *             optional sum_e4 (int64: sum of the e4 codes, the argument of g_b1 = Q_g(e4)) and
 *             acc_dump (int32 accumulators [n,h,w,c_in]).
 */
EOQ_API int eoq_conv_dgrad(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3, const int32_t *e3_exp,
                   const int8_t *w, int8_t *e4, int32_t *e4_exp, int64_t *sum_e4, int32_t *acc_dump,
                   void *workspace, size_t workspace_bytes, void *stream);
/*
 * eoq_conv_dgrad with the error head of the layer that consumes e4 fused into Q_e (what eoq_err_prescale_dev would
 * compute from e4; Sec. 3.2.1, e1 = e0 [x4 > 0], e3 = Q_e(gamma e1) of the layer in front): next_relu_mask, next_x2
 * (optional, int16) and next_gamma (device code) are that layer's; next_e3 (same shape as e4), *next_e3_exp,
 * *next_sum_e1 and (with next_x2) *next_sum_e1x2 are its results.  The GEMM's epilogue reduces the maximum over the
 * positions that layer's ReLU lets through beside the plain one (Q_e is monotonic in |.|, so the largest code of e1 is
 * the code of that maximum), and the pass that writes e4 writes next_e3 as well.  Bit-identical to the two calls in
 * sequence.  EOQ_ERR_UNSUPPORTED for strided 1x1 filters (their sums are kept compact).
 */
EOQ_API int eoq_conv_dgrad_head(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3, const int32_t *e3_exp,
                        const int8_t *w, int8_t *e4, int32_t *e4_exp, int64_t *sum_e4, const uint8_t *next_relu_mask,
                        const int16_t *next_x2, const int32_t *next_gamma, int8_t *next_e3, int32_t *next_e3_exp,
                        int64_t *next_sum_e1, int64_t *next_sum_e1x2, void *workspace, size_t workspace_bytes, void *stream);
/*
 * eoq_conv_dgrad followed by the error join that takes e4 as its first operand (eoq_aux_join: out = Q_e(e4 + b), b
 * gated by mask_b when given) and, when next_relu_mask is not NULL, by the error head of the layer that consumes `out`
 * (eoq_aux_join_head's arguments).  Three kernels instead of five: the join's first pass (its two maxima) rides on the
 * Q_e pass that writes e4.  Bit-identical to the separate calls.  EOQ_ERR_UNSUPPORTED for strided 1x1 filters.
 */
EOQ_API int eoq_conv_dgrad_join_head(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3, const int32_t *e3_exp,
                             const int8_t *w, int8_t *e4, int32_t *e4_exp, int64_t *sum_e4, const int8_t *b, const int32_t *b_exp,
                             const uint8_t *mask_b, int8_t *out, int32_t *out_exp, int64_t *sum_out,
                             const uint8_t *next_relu_mask, const int16_t *next_x2, const int32_t *next_gamma, int8_t *next_e3,
                             int32_t *next_e3_exp, int64_t *next_sum_e1, int64_t *next_sum_e1x2, void *workspace,
                             size_t workspace_bytes, void *stream);

/*
 * eoq_conv_dgrad without any allocation (the paper has no counterpart; this is a deployment variant).
 * Some callers may not allocate device memory at all: code running inside a memory pool that owns the whole
 * device, a plugin loaded into a host application that forbids cudaMalloc after start-up, or a real-time loop
 * where an allocation's implicit synchronisation is not acceptable.  Such callers cannot use eoq_create (it
 * allocates the handle's device state) nor supply a workspace.  This entry point needs neither: every byte of
 * scratch -- reduction cells, transposed weights, int32 sums -- sits in one static device array of
 * EOQ_STATIC_SCRATCH_BYTES (+4 KiB of cells) that is part of the library image, so each GPU that loads the
 * library carries it until the process exits.  It calls no cudaMalloc, cudaFree or allocating library routine.
 *
 * Arguments and results are those of eoq_conv_dgrad (same kernels, bit-identical outputs); there is no handle,
 * no workspace and no acc_dump.  status_out (device, optional) receives the EOQ_DEV_* bits of this call.
 * Limits and rules:
 *   - geometries whose eoq_workspace_size(desc, EOQ_PASS_DGRAD) exceeds EOQ_STATIC_SCRATCH_BYTES are rejected
 *     with EOQ_ERR_WORKSPACE and nothing is launched;
 *   - the first call on a device resolves the array's device address and reads device attributes; make that first
 *     call outside any stream capture, with the device current.  The call itself allocates nothing, but the array's
 *     memory is reserved by the CUDA driver when the library's module is loaded on the device, which happens at the
 *     latest during this first call: on a device whose memory is already taken (a pool that grabbed all of it
 *     before the library was touched) the call returns EOQ_ERR_CUDA, and eoq_last_cuda_error(NULL) gives the
 *     driver's code.  Load the library, and make one call, before handing the device's memory to a pool;
 *   - all calls on a device share the one array, which keeps the previous call's contents: the cells that must
 *     start at zero are cleared on the stream at the start of each call, and two calls that overlap on the GPU
 *     (different streams, no ordering between them) race on it -- order them.
 */
#define EOQ_STATIC_SCRATCH_BYTES (16u << 20)
EOQ_API int eoq_conv_dgrad_static(const eoq_conv_desc_t *desc, const int8_t *e3, const int32_t *e3_exp, const int8_t *w,
                          int8_t *e4, int32_t *e4_exp, int64_t *sum_e4, uint32_t *status_out, void *stream);

/*
 * Weight gradient (Sec. 3.2.1, third equation block): g_w = Q_g(e3 * x1), the correlation of the
 * error with x1 = x0 + Q_b(b1) (zero halo), summed exactly over batch and space, followed by SQ.
 * device in : e3 and *e3_exp as above; x = x0 [n,h,w,c_in] int8.   host in: b1_c.
 * device out: g [c_out,kh,kw,c_in] int8; *g_exp; optional acc_dump (int64, same shape as g).
 */
EOQ_API int eoq_conv_wgrad(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3, const int32_t *e3_exp,
                   const int8_t *x, int32_t b1_c, int8_t *g, int32_t *g_exp, int64_t *acc_dump,
                   void *workspace, size_t workspace_bytes, void *stream);

/* eoq_conv_wgrad with b1 read from device memory (one int32 code; NULL = the layer has no bias before its
 * convolution).  No accumulator dump.  See eoq_conv_fwd_dev. */
EOQ_API int eoq_conv_wgrad_dev(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3, const int32_t *e3_exp,
                       const int8_t *x, const int32_t *b1_c, int8_t *g, int32_t *g_exp, void *workspace,
                       size_t workspace_bytes, void *stream);
/*
 * The weight gradient in two parts, for training loops that finish the gradients of all layers together.
 * eoq_conv_wgrad_gemm: the GEMM of eoq_conv_wgrad_dev alone; the exact sums stay in `workspace` (which must then stay
 *   untouched until the finish) and *num_parts (host) receives what the finish needs to read them.
 * eoq_wgrad_finish: for `num` layers at once (host arrays of length num; device pointers inside): the b1 error sums
 *   (b1_c[i]: the layer's code in device memory, or NULL for a layer without a bias in front of its convolution), the
 *   sum of the split-K slices plus the b1 term, and Q_g -> gq[i], *g_exp[i].  Four launches per 16 layers instead of
 *   four per layer.  workspace[i], workspace_bytes[i], num_parts[i]: as given to / returned by eoq_conv_wgrad_gemm
 *   for that layer; descs[i], e3[i], e3_exp[i] likewise.  Results are those of eoq_conv_wgrad_dev, bit for bit.
 * EOQ_ERR_UNSUPPORTED while a reduce hook is installed (replicas exchange per layer).
 */
EOQ_API int eoq_conv_wgrad_gemm(eoq_handle_t handle, const eoq_conv_desc_t *desc, const int8_t *e3, const int32_t *e3_exp,
                        const int8_t *x, void *workspace, size_t workspace_bytes, int *num_parts, void *stream);
EOQ_API int eoq_wgrad_finish(eoq_handle_t handle, int num, const eoq_conv_desc_t *descs, const int8_t *const *e3,
                     const int32_t *const *e3_exp, const int32_t *const *b1_c, int8_t *const *gq, int32_t *const *g_exp,
                     void *const *workspace, const size_t *workspace_bytes, const int *num_parts, void *stream);

/*
 * The three quantization functions (Sec. 3.2.2) on a flat tensor of n elements.
 *   src_is_float = 1: src is fp32.  Q -> int16 codes R(x * 2^7) (saturated to int16);
 *                     CQ -> int8 codes in [-127,127]; SQ -> int8 codes and *dst_exp.
 *   src_is_float = 0: src is int32 codes with exponent *src_exp (device); only SQ is defined:
 *                     int8 codes and *dst_exp = *src_exp + t - 7.
 * dst_exp may be NULL for Q and CQ.  Uses no workspace (pass NULL, 0).
 */
EOQ_API int eoq_quantize(eoq_handle_t handle, int mode, const void *src, int src_is_float, const int32_t *src_exp,
                 size_t n, void *dst, int32_t *dst_exp, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Head of the error chain (Sec. 3.2.1): e1 = e0 * [x4 > 0], e2 = e1, e3 = Q_e(e2 * Q_gamma(gamma)),
 * with the sums behind g_b2 = Q_g(sum e1) and g_gamma = Q_g(sum e2 * x2).
 * device in : e0 (int8, n_el elements) with exponent *e0_exp; relu_mask as written by eoq_conv_fwd
 *             (NULL = all ones); x2 int16 or NULL.   host in: gamma_c.
 * device out: e3 int8, *e3_exp = *e0_exp - 7 + t - 7; optional sum_e1, sum_e1x2 (int64).
 * n_el must be a multiple of 16.
 */
EOQ_API int eoq_err_prescale(eoq_handle_t handle, const int8_t *e0, const int32_t *e0_exp, const uint8_t *relu_mask,
                     const int16_t *x2, size_t n_el, int32_t gamma_c, int8_t *e3, int32_t *e3_exp,
                     int64_t *sum_e1, int64_t *sum_e1x2, void *stream);

/* eoq_err_prescale with gamma read from device memory (one int32 code, required).  See eoq_conv_fwd_dev. */
EOQ_API int eoq_err_prescale_dev(eoq_handle_t handle, const int8_t *e0, const int32_t *e0_exp, const uint8_t *relu_mask,
                         const int16_t *x2, size_t n_el, const int32_t *gamma_c, int8_t *e3, int32_t *e3_exp,
                         int64_t *sum_e1, int64_t *sum_e1x2, void *stream);

/*
 * The 8-bit update (Sec. 3.2.3, update quantization) on `num` weight tensors in one call:
 *   u = Q_u(lr * g) = SQ(lr * g, 8), lr = lr_mant * 2^lr_exp, lr_mant in [1, 255];
 *   w <- Q_w(w - u): code = sat(R((w - u) * 2^7), -127, 127), in place on the int8 codes.
 * host in   : arrays (host memory, num entries) of device pointers w[i], g[i], g_exp[i] and sizes n[i].
 * EOQ_ROUND_STOCHASTIC (an extension, not in the paper) replaces R by floor((v + r) / 2^s) with r
 * drawn from a counter hash of (seed, step, tensor index, element index).  num <= 256 per call.
 */
EOQ_API int eoq_update(eoq_handle_t handle, int num, int8_t *const *w, const int8_t *const *g,
               const int32_t *const *g_exp, const size_t *n, int32_t lr_mant, int32_t lr_exp, int round_mode,
               uint64_t seed, uint64_t step, void *stream);

/* eoq_update with the step counter in device memory (one uint64, 8-byte aligned): the update reads *step and the
 * call increments it on the device afterwards, so that every replay of a captured step draws fresh rounding bits. */
EOQ_API int eoq_update_dev(eoq_handle_t handle, int num, int8_t *const *w, const int8_t *const *g,
                   const int32_t *const *g_exp, const size_t *n, int32_t lr_mant, int32_t lr_exp, int round_mode,
                   uint64_t seed, uint64_t *step, void *stream);

/*
 * The update at other widths (Sec. 3.2.3 sets the paper's 8-bit update against the 24-bit update of earlier integer
 * training): u = Q_u(lr g) = SQ(lr g, k_u) and a master copy of the weights on the grid of Q(., k_m),
 *   master <- CQ(master - u, k_m)      (int32 codes at exponent -(k_m - 1), updated in place),
 *   w      <- Q_w(master) = code sat(R(master / 2^(k_m - 8)), -127, 127)   (what the layer's three passes read).
 * k_u in [2, 24], k_m in [8, 24]; k_u = k_m = 8 is eoq_update.  Arrays as in eoq_update plus master[i] (device int32,
 * n[i] codes).  step_dev (optional) as in eoq_update_dev, else the host value `step`.
 */
EOQ_API int eoq_update_wide(eoq_handle_t handle, int num, int32_t *const *master, int8_t *const *w, const int8_t *const *g,
                    const int32_t *const *g_exp, const size_t *n, int32_t lr_mant, int32_t lr_exp, int k_u, int k_m,
                    int round_mode, uint64_t seed, uint64_t step, uint64_t *step_dev, void *stream);

/*
 * Input quantizer for the network input (Sec. 5.1 quantizes every layer but the last): SQ(., 8) of an fp32
 * NHWC image batch [n][h][w][c_src], written as int8 [n][h][w + 2 wmargin][c_dst] with c_dst >= c_src: the extra
 * channels and the wmargin pixels at both ends of every row are zero (see eoq_conv_desc_t::x_wmargin).
 * c_dst is 8 or a multiple of 16 and at most 64.  The maximum runs over the whole batch.  *dst_exp is written.
 */
EOQ_API int eoq_quantize_image(eoq_handle_t handle, const float *src, int n, int h, int w, int c_src, int c_dst,
                       int wmargin, int8_t *dst, int32_t *dst_exp, void *stream);

/* int8 layout change between NCHW and NHWC ([n,c,h,w] <-> [n,h,w,c]); to_nhwc = 1 reads NCHW. */
EOQ_API int eoq_layout_convert(eoq_handle_t handle, const int8_t *src, int8_t *dst, int n, int c, int h, int w,
                       int to_nhwc, void *stream);

/*
 * Glue between the layer units of a residual network (the paper chains the units in Sec. 3.2.1 -- x0 of a layer is
 * x5 of the one before, e0 the error its successor hands back -- and keeps the last layer in floating point,
 * Sec. 5.1; pooling, the shortcut error and the float arithmetic are not specified there and follow the conventions
 * stated with each call).  All tensors NHWC, channel counts multiples of 16, pointers device unless noted.
 */

/* Max-pooling of int8 codes, window k x k: y [n,ho,wo,c]; arg (same shape, uint8) = kh * k + kw of the first maximum in
 * (kh, kw) scan order (padding never wins). */
EOQ_API int eoq_aux_maxpool_fwd(eoq_handle_t handle, const int8_t *x, int n, int h, int w, int c, int k, int stride, int pad,
                        int8_t *y, uint8_t *arg, void *stream);
/* Its backward: every error code e [n,ho,wo,c] (exponent *e_exp) is added at the position its window elected, the
 * exact sums are requantized with Q_e = SQ: e_in [n,h,w,c], *e_in_exp. */
EOQ_API int eoq_aux_maxpool_bwd(eoq_handle_t handle, const int8_t *e, const int32_t *e_exp, const uint8_t *arg, int n, int h, int w,
                        int c, int k, int stride, int pad, int8_t *e_in, int32_t *e_in_exp, void *stream);
/* The same with the error head of the layer in front of the pool fused in (what eoq_err_prescale_dev would compute
 * from e_in, without x2): e1 = e_in * [x4 > 0] (relu_mask of that layer, bit i of the NHWC element index),
 * e3 = Q_e(gamma * e1) [n,h,w,c] with *e3_exp, *sum_e1 (optional) = sum of the e1 codes; gamma: that layer's code in
 * device memory.  e_in and e_in_exp may be NULL when only e3 is wanted.  Bit-identical to the two calls in sequence. */
EOQ_API int eoq_aux_maxpool_bwd_head(eoq_handle_t handle, const int8_t *e, const int32_t *e_exp, const uint8_t *arg, int n, int h,
                             int w, int c, int k, int stride, int pad, int8_t *e_in, int32_t *e_in_exp,
                             const uint8_t *relu_mask, const int32_t *gamma, int8_t *e3, int32_t *e3_exp, int64_t *sum_e1,
                             void *stream);
/* Global average pooling hands exact integer sums to the head: sums[n][c] = sum over the hw positions of x. */
EOQ_API int eoq_aux_avgpool_sum(eoq_handle_t handle, const int8_t *x, int n, int hw, int c, int32_t *sums, void *stream);
/*
 * Where the error of a residual branch (a, exponent *a_exp) meets the error arriving through the shortcut (b,
 * *b_exp; gated by mask_b, bit-packed as eoq_conv_fwd writes it, NULL = no gate): both are brought to the smaller
 * exponent, added exactly (an operand more than 31 octaves below the other is dropped) and requantized with
 * Q_e = SQ over the whole tensor.  out, *out_exp; sum_out (optional) = sum of the out codes (for g_b1).
 * n_el a multiple of 16.
 */
EOQ_API int eoq_aux_join(eoq_handle_t handle, const int8_t *a, const int32_t *a_exp, const int8_t *b, const int32_t *b_exp,
                 const uint8_t *mask_b, size_t n_el, int8_t *out, int32_t *out_exp, int64_t *sum_out, void *stream);
/* The same with the error head of the layer that consumes `out` fused in (what eoq_err_prescale_dev would compute from
 * out): e1 = out * [x4 > 0] (relu_mask of that layer), e3 = Q_e(gamma * e1) with *e3_exp, *sum_e1 and, when x2 is given
 * (int16, that layer's x2), *sum_e1x2 = sum of e1 * x2; gamma: that layer's code in device memory.  Bit-identical to
 * the two calls in sequence. */
EOQ_API int eoq_aux_join_head(eoq_handle_t handle, const int8_t *a, const int32_t *a_exp, const int8_t *b, const int32_t *b_exp,
                      const uint8_t *mask_b, size_t n_el, int8_t *out, int32_t *out_exp, int64_t *sum_out,
                      const uint8_t *relu_mask, const int16_t *x2, const int32_t *gamma, int8_t *e3, int32_t *e3_exp,
                      int64_t *sum_e1, int64_t *sum_e1x2, void *stream);
/*
 * The floating-point last layer, operation by operation in fp32 (every product-sum is one fused multiply-add, sums
 * run over ascending indices into one accumulator, exp is a fixed polynomial), so that any IEEE-754 machine gives
 * the same bits: pooled = (float)sums * 2^-7 / hw; logits = W pooled + bias (W [classes][c]); softmax cross-entropy,
 * mean over the batch; dpooled [n][c] = its gradient with respect to pooled (W before the update); W and bias take
 * one SGD step with rate lr, in place.  *loss (optional) is reported only (its logarithm is the library's).
 * labels int32 [n].  workspace: eoq_aux_head_workspace_size bytes, 256-byte aligned.
 */
EOQ_API int eoq_aux_head_workspace_size(int n, int c, int classes, size_t *bytes);
EOQ_API int eoq_aux_head(eoq_handle_t handle, const int32_t *sums, int n, int c, int hw, int classes, float *W, float *bias,
                 const int32_t *labels, float lr, float *loss, float *dpooled, float *logits, void *workspace,
                 size_t workspace_bytes, void *stream);
/* The SGD step of W and bias alone, from what the last eoq_aux_head call on this workspace left there (its pooled
 * activations and logit gradients): for callers that pass lr = 0 to eoq_aux_head (W and bias then stay untouched,
 * which is what a zero rate means) and take the step later, e.g. on another stream beside the backward pass.
 * The results are the ones eoq_aux_head gives with that lr. */
EOQ_API int eoq_aux_head_update(eoq_handle_t handle, int n, int c, int classes, float *W, float *bias, float lr, const void *workspace,
                        size_t workspace_bytes, void *stream);
/* The error the head hands back: SQ over all of dpooled / hw (the gradient of one position of the average), the
 * code of (sample, channel) written to all hw positions: e [n][hw][c], *e_exp.  workspace: n*c floats. */
EOQ_API int eoq_aux_head_error(eoq_handle_t handle, const float *dpooled, int n, int c, int hw, int8_t *e, int32_t *e_exp,
                       void *workspace, size_t workspace_bytes, void *stream);
/*
 * Comparison case, not on the EOQ path (Sec. 5.3 sets the Fixup scale and bias against "traditional BN"): training-
 * mode batch normalisation of a convolution output, per channel over all `pixels` = n*ho*wo positions of the batch.
 *   acc      [pixels][c] exact int32 sums of the convolution (the acc_out of eoq_conv_fwd) at exponent acc_exp
 *            (-14 for int8 codes at -7 times int8 weights at -7); c a multiple of 16, at most 1024.
 *   gamma, beta  fp32 [c] (device).  eps added to the biased variance.
 * eoq_bn_fwd: y = gamma (a - mean) / sqrt(var + eps) + beta; x5 = Q_a2(relu(y)) int8 codes at exponent -7;
 *   relu_mask bit = [y > 0].  The statistics are exact integer sums; the per-channel constants are formed in double
 *   precision and each element takes one fp32 fused multiply-add, so the result is reproducible bit for bit.
 * eoq_bn_bwd: for error codes e at exponent *e_exp arriving at x5 (same shape), dy = e * mask:
 *   dgamma, dbeta fp32 [c]; da fp32 [pixels][c] = the error with respect to the convolution output (quantize it with
 *   eoq_quantize(EOQ_SQ) to obtain the int8 error the dgrad and wgrad passes take).  Must follow eoq_bn_fwd on the
 *   same workspace (it reads the statistics left there).
 * workspace: eoq_bn_workspace_size(c) bytes, 256-byte aligned, owned by the caller.
 * Errors: EOQ_ERR_BAD_ARG (null pointer, pixels == 0), EOQ_ERR_ALIGNMENT (c % 16, unaligned pointers),
 * EOQ_ERR_UNSUPPORTED (c > 1024), EOQ_ERR_WORKSPACE.
 */
EOQ_API int eoq_bn_workspace_size(int c, size_t *bytes);
EOQ_API int eoq_bn_fwd(eoq_handle_t handle, const int32_t *acc, int acc_exp, size_t pixels, int c, const float *gamma,
               const float *beta, float eps, int8_t *x5, uint8_t *relu_mask, void *workspace, size_t workspace_bytes,
               void *stream);
EOQ_API int eoq_bn_bwd(eoq_handle_t handle, const int8_t *e, const int32_t *e_exp, const uint8_t *relu_mask, const int32_t *acc,
               int acc_exp, size_t pixels, int c, const float *gamma, void *workspace, size_t workspace_bytes, float *da,
               float *dgamma, float *dbeta, void *stream);
/*
 * Update of `num` scalar parameters (gamma, b1, b2; Sec. 3.2.3 applied to a single value): g = Q_g({total}) with
 * total the exact sum behind the gradient at exponent *total_exp[i] + exp_bias[i]; u = Q_u(lr g);
 * theta <- Q(theta - u) saturated to 16 bits, rounding as in eoq_update (the hash counter of scalar i is
 * tensor_id[i], element 0).  Host arrays of device pointers: theta[i] (int32 code, updated in place), mirror[i]
 * (optional second copy), total[i] (int64), total_exp[i] (int32), grad_out[i] (optional, receives {code, exponent} of
 * g).  step: device step counter as in eoq_update_dev (read, not incremented) or NULL for 0.
 */
EOQ_API int eoq_aux_scalar_update(eoq_handle_t handle, int num, int32_t *const *theta, int32_t *const *mirror,
                          const int64_t *const *total, const int32_t *const *total_exp, const int *exp_bias,
                          const int *tensor_id, int32_t *const *grad_out, int32_t lr_mant, int32_t lr_exp, int round_mode,
                          uint64_t seed, const uint64_t *step, void *stream);

/* Synchronises `stream`, returns the OR of the EOQ_DEV_* bits raised since the last call, clears them. */
EOQ_API int eoq_last_status(eoq_handle_t handle, void *stream, unsigned *bits);

/*
 * Instrumentation (off by default).  Between eoq_profile_start and eoq_profile_stop the kernels of each call are
 * bracketed by CUDA events on their stream, grouped in EOQ_PROF_KINDS kinds.  eoq_profile_stop synchronises the
 * device and reports per kind the number of bracketed groups and their summed duration in milliseconds; it keeps
 * at most 8192 groups.  eoq_launch_count returns how many kernels this handle has launched so far.
 */
#define EOQ_PROF_IGEMM_FWD 0     /* the forward implicit-GEMM kernel, one launch per group */
#define EOQ_PROF_IGEMM_DGRAD 1   /* the dgrad implicit-GEMM kernel, one launch per group */
#define EOQ_PROF_WGRAD 2         /* the weight-gradient GEMM kernel */
#define EOQ_PROF_ERR_HEAD 3      /* eoq_err_prescale (one kernel; two for tensors beyond the one-kernel capacity) */
#define EOQ_PROF_DGRAD_AUX 4     /* Q_e phase 2; weight transpose (only layers with fewer than 32 output channels) */
#define EOQ_PROF_WGRAD_AUX 5     /* slice sum + b1 term + Q_g behind the weight-gradient GEMM (and the memset in front of it) */
#define EOQ_PROF_FWD_AUX 6       /* b1 weight table, weight row padding (eoq_weight_prep, or per call without it) */
#define EOQ_PROF_OTHER 7         /* eoq_quantize, eoq_bn_fwd, eoq_bn_bwd */
#define EOQ_PROF_UPDATE 8        /* eoq_update */
#define EOQ_PROF_INPUT_Q 9       /* eoq_quantize_image */
#define EOQ_PROF_WGRAD_TAPS 10   /* b1 error sums of the weight gradient */
#define EOQ_PROF_GLUE 11         /* eoq_aux_*: pooling, error join, float head, scalar updates */
#define EOQ_PROF_KINDS 12
EOQ_API int eoq_profile_start(eoq_handle_t handle);
EOQ_API int eoq_profile_stop(eoq_handle_t handle, int launches[EOQ_PROF_KINDS], double milliseconds[EOQ_PROF_KINDS]);
EOQ_API unsigned long long eoq_launch_count(eoq_handle_t handle);
/* Timing aid: while on, eoq_conv_dgrad and eoq_conv_wgrad (and their _dev forms) on this handle launch their GEMM
 * kernel only -- no quantizer behind it, no helper in front -- so the outputs of those calls are NOT produced; used
 * to time the tensor-core kernels alone, back to back.  Synchronises the device; switching it off puts the handle's
 * reduction cells back to zero. */
EOQ_API int eoq_profile_gemm_only(eoq_handle_t handle, int on);

/*
 * Data-parallel replicas (the paper trains with synchronous SGD on several GPUs, Sec. 5.1).  Every quantizer of the
 * layer that reduces over the batch -- the maximum behind each SQ (Sec. 3.2.2), the sums behind the scalar gradients,
 * the exact weight-gradient sums in front of Q_g (Sec. 3.2.1) -- forms its value in one kernel and consumes it in a
 * later one.  With a hook set, the library calls it on the host between the two, with the device buffer that holds
 * the local value; the hook enqueues an all-reduce of that buffer on `stream` (ncclAllReduce or the like: in place,
 * `count` elements, dtype EOQ_REDUCE_I32 or EOQ_REDUCE_I64, op EOQ_REDUCE_MAX over non-negative values or
 * EOQ_REDUCE_SUM).  Replicas that each hold a share of the batch then continue with the global value and write, bit
 * for bit, what one device writes on the whole batch: integer maxima and sums do not depend on the order of
 * reduction.  (One-kernel forms of a call give way to their two-kernel forms while a hook is set.  The float last
 * layer reduces in a fixed order over the samples: replicas gather sums and labels and each runs eoq_aux_head on
 * the whole batch.)  fn = NULL removes the hook.
 */
#define EOQ_REDUCE_I32 0
#define EOQ_REDUCE_I64 1
#define EOQ_REDUCE_MAX 0
#define EOQ_REDUCE_SUM 1
typedef void (*eoq_reduce_fn)(void *user, void *device_buffer, size_t count, int dtype, int op, void *stream);
EOQ_API int eoq_set_reduce_hook(eoq_handle_t handle, eoq_reduce_fn fn, void *user);

/* Caps the CTAs (one per SM) that the GEMM launches of this handle use; 0 = one per SM of the device (the
 * default).  Every GEMM kernel is persistent: with fewer CTAs a launch walks more tiles per CTA and leaves the
 * other SMs free, so that GEMMs issued through two handles on two streams run side by side instead of one after
 * the other (in the training step of Sec. 3.2.1 the error back-propagation of a layer and its weight gradient are
 * independent once e3 exists).  Results do not depend on the setting.  Host-side state only; applies to the calls
 * made after it. */
EOQ_API int eoq_set_gemm_ctas(eoq_handle_t handle, int ctas);

/*
 * Measures what the tensor pipe delivers for the instruction all three convolution passes run on, tcgen05.mma
 * kind::i8 with a 128 x n_cols x 32 shape (int8 x int8 -> int32, Sec. 3.2.1): one CTA per SM, operands resident in
 * shared memory, two accumulators in tensor memory, `iters` x 4 MMAs per CTA and launch, `launches` launches timed
 * with CUDA events on `stream`.  Synchronises.  *tops = operations (2 per multiply-add) per second / 1e12 over the
 * timed launches, launch gaps included; *cycles_per_mma (optional) = SM clock cycles per MMA inside the longest
 * issue loop.  n_cols: a multiple of 16 in [16, 256].  A measurement aid for roofline denominators, not part of
 * the layer.
 */
EOQ_API int eoq_probe_mma_i8(eoq_handle_t handle, int n_cols, int iters, int launches, double *tops, double *cycles_per_mma,
                     void *stream);

/* One line of text saying which kernel and tiling a pass of this geometry takes on this handle (for tests and
 * reports; the format is not an interface).  buf receives at most buf_bytes bytes, NUL-terminated. */
EOQ_API int eoq_describe_plan(eoq_handle_t handle, const eoq_conv_desc_t *desc, int pass, char *buf, size_t buf_bytes);

/* Self-test of the bounded device waits: the next eoq_err_prescale / eoq_err_prescale_dev call on this handle that
 * takes the one-kernel path waits at its grid-wide barrier for one block more than exists, with a limit of 2048
 * polls (about 0.2 ms).  The wait runs out, the kernel raises EOQ_DEV_TIMEOUT, writes no output and returns;
 * eoq_last_status then reports the bit and puts the handle's reduction cells back to zero.  Nothing faults or
 * hangs; one call only, then the handle behaves normally again. */
EOQ_API int eoq_debug_force_wait_timeout(eoq_handle_t handle);

/* The last cudaError_t a call on this handle recorded (0 if none); handle = NULL: the last one of
 * eoq_conv_dgrad_static, which has no handle. */
EOQ_API int eoq_last_cuda_error(eoq_handle_t handle);

EOQ_API const char *eoq_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* EOQ_H */
