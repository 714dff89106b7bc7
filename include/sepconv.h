/*
 * sepconv.h -- C ABI of the B200 (sm_100a) time-channel separable convolution library.
 *
 * The library computes the forward and backward pass of the block that makes up a
 * Jasper/QuartzNet-style convolutional acoustic encoder, the `JasperEncoder` neural module of
 * the NeMo paper (arXiv 1909.09577, section 4.1.1), whose ports are
 *     (audio_signal [B, C, T], length [B])  ->  (encoded [B, C', T'], encoded_len [B]).
 * Tensors are described the way the paper's neural types describe them (section 3.2, Table 1):
 * every axis carries a semantic tag (batch / channel / time) and a size, and a mismatch is
 * reported with the same vocabulary (dimension-incompatible, transposed, incompatible).
 * Precision follows section 3.3: 16-bit (or fp32) activations and convolution weights, fp32
 * accumulation, statistics, affine parameters and parameter gradients.
 *
 * One layer ("block") computes, for x [B, C_in, T_in] and lengths len[b] (in input frames):
 *     xm = x where t <  len[b], else 0                                   (padding mask)
 *     u[b,c,t]  = sum_k wd[c,k] * xm[b,c,t*stride + k*dilation - P]       (depthwise, zero "same" padding:
 *                 dilation*(K-1) zeros in total, P = floor of half of them on the left)
 *     v[b,o,t]  = sum_c wp[o,c] * u[b,c,t]  (+ bias[o])                   (pointwise 1x1)
 *     len'[b]   = ceil(len[b]/stride);  N = sum_b len'[b]
 *     mean, var = per-channel moments of v over the N valid frames (biased variance)
 *     bn        = gamma * (v - mean) / sqrt(var + eps) + beta            (training-mode batch norm)
 *     r         = 0 | xr (identity) | BN_r(wr * xr)  (projection), xr = residual source masked by len'
 *     y         = relu(bn + r)           (res_before_relu = 1, the default)
 *               = relu(bn) + r           (res_before_relu = 0)
 *     y = 0 for t >= len'[b]
 * and the exact gradient of that map.  A linear layer (has_bn = 0) may end in the decoder's log-softmax over its
 * channels (log_softmax = 1): y[b,:,t] = z[b,:,t] - log(sum_c exp(z[b,c,t])) with z = wp u + bias.  T' = floor((T_in - 1)/stride) + 1.
 *
 * Conventions common to all calls
 *   - Every pointer named *_dev or held in an sc_tensor / sc_block_params / sc_block_saved /
 *     sc_block_grads is a DEVICE pointer owned by the caller; descriptors are HOST structs.
 *   - Tensors are dense [B, C, T] with time contiguous; base pointers 16-byte aligned.
 *   - Activations and conv weights (wd, wp, wr) use desc->io_dtype; gamma, beta, bias, the saved
 *     statistics, running statistics and every parameter gradient are float32.
 *   - Tensors that only the library sees between the depthwise and the pointwise step (u forward;
 *     the gradients of v and u backward) are float16 for both 16-bit activation types: they are
 *     contraction operands, and a second bf16 rounding on them would cost more than the error budget
 *     leaves.  Forward, a depthwise output beyond the float16 range is clamped and reported as
 *     SC_ERR_RANGE; backward, those gradients carry a per-layer power-of-two scale chosen on the
 *     device from the gradient's magnitude, so any upstream scale (e.g. a loss scale) is safe.
 *   - Calls enqueue work on `cuda_stream` and return without synchronising.  The library never
 *     allocates or frees device memory inside these calls and keeps no pointer past the call.
 *   - Return value: SC_OK or a negative sc_status.  Nothing throws across the boundary.  Errors
 *     that only the device can see (a length outside [1, T], a bounded wait that ran out) are
 *     written to a status word that sepconv_last_status() returns.
 *   - Results are deterministic: reductions use a fixed order, no floating-point atomics.
 */
#ifndef SEPCONV_H_
#define SEPCONV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sc_ctx sc_ctx;

typedef enum { SC_F32 = 0, SC_F16 = 1, SC_BF16 = 2 } sc_dtype;
/* semantic axis tags (section 3.2) */
typedef enum { SC_AX_BATCH = 0, SC_AX_CHANNEL = 1, SC_AX_TIME = 2 } sc_axis;
typedef enum { SC_RES_NONE = 0, SC_RES_IDENTITY = 1, SC_RES_PROJ = 2 } sc_residual;

typedef enum {
    SC_OK = 0,
    SC_ERR_NULL = -1,              /* a required pointer is null                                   */
    SC_ERR_INCOMPATIBLE = -2,      /* wrong dtype or rank                                          */
    SC_ERR_DIM_INCOMPATIBLE = -3,  /* an axis size disagrees with the descriptor                   */
    SC_ERR_TRANSPOSED = -4,        /* right sizes, wrong axis order (e.g. [B,T,C]) or not dense    */
    SC_ERR_ALIGNMENT = -5,         /* base pointer not 16-byte aligned                             */
    SC_ERR_UNSUPPORTED = -6,       /* even K, stride not 1|2, illegal residual, ...                */
    SC_ERR_WORKSPACE = -7,         /* workspace too small or null                                  */
    SC_ERR_LENGTHS = -8,           /* (device) some length is outside [1, T_in]                    */
    SC_ERR_DEVICE_TIMEOUT = -9,    /* (device) a bounded wait inside a kernel ran out              */
    SC_ERR_ARCH = -10,             /* the device is not compute capability 10.x                    */
    SC_ERR_CUDA = -11,             /* a CUDA runtime/driver call failed                            */
    SC_ERR_RANGE = -12             /* (device) a depthwise or pointwise result exceeded the float16 range */
} sc_status;

/* A typed tensor argument: size/stride in elements, tag[i] names axis i. */
typedef struct {
    void*   ptr;
    int32_t dtype;      /* sc_dtype */
    int32_t rank;       /* must be 3 */
    int64_t size[3];
    int64_t stride[3];
    int32_t tag[3];     /* sc_axis; the library expects {BATCH, CHANNEL, TIME} */
} sc_tensor;

typedef struct {
    int32_t B, C_in, C_out, T_in;
    int32_t K, stride;          /* K >= 1; stride 1 or 2 (ignored when has_dw = 0).  Odd K with adjacent */
                                /* taps takes the tensor-core depthwise kernels; even K or dilation > 1  */
                                /* takes plain kernels                                                   */
    int32_t io_dtype;           /* sc_dtype of activations and conv weights                        */
    int32_t residual;           /* sc_residual                                                     */
    int32_t C_res;              /* channels of the residual source (0: same as C_in)               */
    int32_t has_dw, has_bn, has_relu, has_bias;
    int32_t res_before_relu;    /* 1: y = relu(bn + r);  0: y = relu(bn) + r                       */
    float   bn_eps, bn_momentum;
    int32_t log_softmax;        /* 1: y = log-softmax over the channels of (wp u + bias), the decoder   */
                                /* module's log_probs (section 4.1.1); only on a layer with has_bn = 0,  */
                                /* has_relu = 0 and no residual.  Backward then takes dL/dlog_probs      */
    int32_t dilation;           /* frames between neighbouring depthwise taps (0 or 1: adjacent)          */
    int32_t full_conv;          /* 1: block variant with ONE non-separable K-tap convolution in place of  */
                                /* depthwise + pointwise (the convolution of the original Jasper block,   */
                                /* section 4.1.1): params.wp is [C_out, C_in, K]; K, stride and dilation   */
                                /* apply to it with the depthwise step's conventions; has_dw must be 0 and */
                                /* log_softmax 0; saved.u is not used.  Plain (non-tensor-core) kernels    */
} sc_block_desc;

typedef struct {          /* device pointers; absent parts may be null                             */
    const void  *wd;      /* [C_in, K]      io_dtype                                               */
    const void  *wp;      /* [C_out, C_in]  io_dtype                                               */
    const float *gamma, *beta;       /* [C_out]                                                    */
    const float *bias;               /* [C_out]                                                    */
    const void  *wr;      /* [C_out, C_res] io_dtype                                               */
    const float *gamma_r, *beta_r;   /* [C_out]                                                    */
} sc_block_params;

typedef struct {          /* written by sepconv_fwd, read by sepconv_bwd; caller-owned             */
    void  *u;             /* [B, C_in, T'] depthwise output (or masked input when has_dw = 0).     */
                          /* float16 when the layer has a depthwise step and batch norm and        */
                          /* io_dtype is 16-bit (also for bf16: see below); io_dtype otherwise     */
    void  *v;             /* [B, C_out, T'] pointwise result before normalisation (has_bn only);   */
                          /* float32 when io_dtype is SC_F32, float16 otherwise (a value beyond    */
                          /* the float16 range is clamped and reported as SC_ERR_RANGE); frames    */
                          /* at and beyond len'[b] are unspecified and never read                  */
    float *mean, *invstd; /* [C_out]                                                               */
    void  *vr;            /* same for the projection residual branch: wr * xr                      */
    float *mean_r, *invstd_r;
} sc_block_saved;

typedef struct {          /* float32 parameter gradients, same shapes as the parameters            */
    float *dwd, *dwp, *dgamma, *dbeta, *dbias, *dwr, *dgamma_r, *dbeta_r;
} sc_block_grads;

/* Encoder = a fixed list of layers.  res_from[i] = index of the layer whose INPUT feeds layer i's
 * residual branch (-1: layer i's own input).  B and T_in of layers[0] are the encoder's; the
 * B/T_in fields of later layers are ignored and derived.  param_offsets / grad_offsets are HOST
 * arrays of n_layers*8 byte offsets (order: wd, wp, gamma, beta, bias, wr, gamma_r, beta_r; -1 for
 * an absent parameter) into the caller's flat device blobs. */
typedef struct {
    int32_t              n_layers;
    const sc_block_desc* layers;
    const int32_t*       res_from;
} sc_encoder_desc;

/* ---- context ------------------------------------------------------------------------------ */

/* Creates a context on CUDA device `device` (which must be compute capability 10.x) and allocates
 * the 64-byte device status word -- the only device allocation the library ever makes.
 * Returns SC_ERR_ARCH on any other architecture.  (The paper's modules are created once by a factory
 * and then only executed, section 3.1; the context is that create-once state: device, status word,
 * resolved driver entry points.) */
int  sepconv_ctx_create(sc_ctx** out, int device);
void sepconv_ctx_destroy(sc_ctx* ctx);

/* Synchronises `cuda_stream`, returns the device status word (SC_OK, SC_ERR_LENGTHS, SC_ERR_RANGE or
 * SC_ERR_DEVICE_TIMEOUT) and clears it.  These are the errors only the device can see: the `length`
 * port of section 4.1.1 holding a value outside [1, T], an intermediate leaving the float16 range that
 * section 3.3's mixed-precision policy stores it in, a bounded wait inside a kernel that ran out. */
int  sepconv_last_status(sc_ctx* ctx, void* cuda_stream);
/* Text for a status code.  The argument-validation codes follow the outcomes of the paper's neural-type
 * comparison (section 3.2): an axis of the wrong size is DIM_INCOMPATIBLE (Table 1's 64- vs 40-channel
 * spectrogram rows), the right axes in the wrong order are TRANSPOSED (the paper's TRANSPOSE_SAME),
 * another element type, rank or set of axis tags is INCOMPATIBLE. */
const char* sepconv_strerror(int status);

/* Launches one small kernel whose only thread waits, with a short poll limit, on a barrier that nothing
 * signals: the wait must run out and leave SC_ERR_DEVICE_TIMEOUT in the status word, and the context
 * must stay usable.  It exercises the give-up path that every device-side wait of the library has
 * (the paper has no counterpart; nothing is left in flight and the GPU is not faulted or hung). */
int  sepconv_selftest_bounded_wait(sc_ctx* ctx, void* cuda_stream);

/* ---- one block ---------------------------------------------------------------------------- */

/* Bytes of scratch the two block calls need for this descriptor (host-only computation).  The block
 * descriptor is the module's constructor arguments as a plain struct: the paper keeps a module's
 * structure in data, not in code (section 3).  Returns SC_ERR_UNSUPPORTED for a descriptor the
 * library does not implement (even K, stride other than 1 or 2, identity residual across a channel
 * change, ...). */
int  sepconv_workspace_bytes(const sc_block_desc* desc, size_t* fwd_bytes, size_t* bwd_bytes);

/* Forward of one block (definition at the top of this file): the body of the encoder module of section
 * 4.1.1, whose ports are (audio_signal, length) -> (encoded, encoded_len); every tensor argument is
 * checked against the [batch, channel, time] neural type of section 3.2 before anything is enqueued.
 *   x              [B, C_in, T_in]
 *   x_res          residual source [B, C_res, T']; null = x (requires stride 1)
 *   lengths_dev    int32 [B], valid input frames, each in [1, T_in]
 *   y              [B, C_out, T'] (written, zero in padded frames)
 *   out_lengths_dev int32 [B] <- len' (nullable)
 *   saved          intermediates for the backward pass (see sc_block_saved)
 *   running_mean/var  float32 [C_out], updated in place with bn_momentum (nullable)
 */
int  sepconv_fwd(sc_ctx* ctx, const sc_block_desc* desc,
                 const sc_tensor* x, const sc_tensor* x_res, const int32_t* lengths_dev,
                 const sc_block_params* params, sc_tensor* y, int32_t* out_lengths_dev,
                 sc_block_saved* saved, float* running_mean, float* running_var,
                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Backward of one block: the exact adjoint of sepconv_fwd.
 *   dy       upstream gradient [B, C_out, T'] (values in padded frames are ignored)
 *   x, x_res, y, lengths_dev, params, saved: as given to / produced by sepconv_fwd
 *   dx       [B, C_in, T_in]  <- gradient w.r.t. x (zero in padded frames)
 *   dx_res   [B, C_res, T']   <- gradient w.r.t. x_res; null = the residual path's gradient is
 *            added into dx (only legal when the residual source is x: with a separate x_res and no
 *            dx_res the call returns SC_ERR_UNSUPPORTED)
 *   dx_add   optional [B, C_in, T_in] tensor added into dx before rounding (a gradient that
 *            reaches the same input along another path)
 *   grads    parameter gradients, float32; accumulate != 0 adds into them instead of overwriting
 *            (gradient accumulation, section 3.3)
 */
int  sepconv_bwd(sc_ctx* ctx, const sc_block_desc* desc,
                 const sc_tensor* dy, const sc_tensor* x, const sc_tensor* x_res, const sc_tensor* y,
                 const int32_t* lengths_dev, const sc_block_params* params,
                 const sc_block_saved* saved,
                 sc_tensor* dx, sc_tensor* dx_res, const sc_tensor* dx_add,
                 sc_block_grads* grads, int accumulate,
                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Evaluation-mode forward of one block (the paper's `eval` / `infer` actions, section 3.1): batch statistics are
 * replaced by the given running statistics,  bn = gamma (v - running_mean) / sqrt(running_var + eps) + beta,
 * everything else as in sepconv_fwd; nothing is saved for a backward pass and the running statistics are
 * only read.  running_mean_r / running_var_r belong to the projection residual's batch norm (null otherwise).
 * Scratch: sepconv_infer_workspace_bytes. */
int  sepconv_infer_workspace_bytes(const sc_block_desc* desc, size_t* bytes);
int  sepconv_infer(sc_ctx* ctx, const sc_block_desc* desc,
                   const sc_tensor* x, const sc_tensor* x_res, const int32_t* lengths_dev,
                   const sc_block_params* params,
                   const float* running_mean, const float* running_var,
                   const float* running_mean_r, const float* running_var_r,
                   sc_tensor* y, int32_t* out_lengths_dev,
                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Forward of one block without a workspace argument and without any allocation (the paper has no
 * counterpart; this exists for integration reasons only).
 *
 * Who needs it: code that runs where device allocation is forbidden or impossible -- inside a
 * real-time audio pipeline whose memory is fixed at start-up, under a framework that owns the whole
 * device heap and hands out no raw buffers, or in a plugin loaded after the host application has
 * already committed all device memory.  Such a caller can still pass its own inputs and outputs but
 * has nowhere to get the scratch that sepconv_fwd asks for.
 *
 * The scratch is a fixed array of SEPCONV_STATIC_SCRATCH_BYTES inside the library image: every GPU on
 * which the library is loaded sets that much memory aside until the process exits.  A block whose
 * forward scratch (sepconv_workspace_bytes) exceeds it is refused with SC_ERR_WORKSPACE and a message
 * on stderr; nothing is enqueued.  Arguments and results are exactly those of sepconv_fwd (running
 * statistics are not updated).  The call itself uses no cudaMalloc/cudaFree or other allocating
 * routine.
 *
 * The first call on each device looks up the array's device address; with CUDA's lazy module loading
 * that is also the moment the device sets the array aside, so this first call can still fail with
 * SC_ERR_CUDA on a device whose memory is already fully committed: make it once at start-up, outside
 * any stream capture.  The context's device must be the current device (SC_ERR_UNSUPPORTED otherwise:
 * the array belongs to the current device).
 * All calls on a device share the one array and it keeps the previous call's contents: two calls
 * whose GPU work overlaps (different streams, no dependency between them) race on it -- keep such
 * calls on one stream or order them with events. */
#define SEPCONV_STATIC_SCRATCH_BYTES (8u << 20)
int  sepconv_fwd_static(sc_ctx* ctx, const sc_block_desc* desc,
                        const sc_tensor* x, const sc_tensor* x_res, const int32_t* lengths_dev,
                        const sc_block_params* params, sc_tensor* y, int32_t* out_lengths_dev,
                        sc_block_saved* saved, void* cuda_stream);

/* ---- whole encoder -------------------------------------------------------------------------- */

/* Bytes of workspace encoder_fwd_bwd needs for this layer list (host-only computation).  A layer's residual
 * may come from the input of any earlier layer (res_from[i] <= i; a later one: SC_ERR_UNSUPPORTED); the spans
 * [res_from[i], i] may nest or overlap and several layers may name the same source.  The residual path's gradient
 * for a source waits in a pending buffer until the backward pass reaches that source; spans that do not overlap
 * share one buffer (the Jasper-style encoders of section 4.1.1, where each block's residual comes from that block's
 * input, need a single one), each overlapping span adds a buffer of the source's size to the workspace.  One
 * residual source per layer: the sum of several projected sources at one layer (the dense-residual variant of the
 * Jasper family) is not expressible. */
int  encoder_workspace_bytes(const sc_encoder_desc* desc, size_t* bytes);

/* The whole encoder module of section 4.1.1 plus the 1x1 decoder convolution that ends in the logits
 * (`jasper_encoder` then `jasper_decoder` without its log-softmax): forward through every layer, then
 * backward from `dlogits`, in one call.
 *   x [B, C_0, T_in], lengths_dev int32 [B]
 *   params_blob / grads_blob: flat device blobs addressed by param_offsets / grad_offsets
 *   dlogits [B, C_last, T_last] upstream gradient; logits [B, C_last, T_last] (written)
 *   out_lengths_dev int32 [B] <- encoded lengths;  dx (nullable) <- gradient w.r.t. x
 * All per-layer intermediates live in `workspace`.
 */
int  encoder_fwd_bwd(sc_ctx* ctx, const sc_encoder_desc* desc,
                     const sc_tensor* x, const int32_t* lengths_dev,
                     const void* params_blob, const int64_t* param_offsets,
                     const sc_tensor* dlogits, sc_tensor* logits, int32_t* out_lengths_dev,
                     void* grads_blob, const int64_t* grad_offsets, sc_tensor* dx,
                     int accumulate, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Evaluation-mode forward through every layer (sepconv_infer per layer, intermediates in `workspace`):
 *   running_blob / running_offsets: flat device blob of float32 running statistics and a HOST array of
 *   n_layers*4 byte offsets (order: mean, var, mean_r, var_r; -1 where the layer has none)
 *   out [B, C_last, T_last] <- logits, or log_probs when the last layer has log_softmax = 1. */
int  encoder_infer_workspace_bytes(const sc_encoder_desc* desc, size_t* bytes);
int  encoder_infer(sc_ctx* ctx, const sc_encoder_desc* desc,
                   const sc_tensor* x, const int32_t* lengths_dev,
                   const void* params_blob, const int64_t* param_offsets,
                   const void* running_blob, const int64_t* running_offsets,
                   sc_tensor* out, int32_t* out_lengths_dev,
                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Selects the kernel family for the pointwise contractions: 0 = automatic (tensor cores where
 * the shape allows), 1 = force the plain fp32-accumulate SIMT kernels.  Used by tests (the paper has
 * no counterpart). */
int  sepconv_set_gemm_mode(sc_ctx* ctx, int mode);

/* Tile shape of the forward / input-gradient pointwise contractions (tuning aid; the paper has no counterpart):
 * 0 = 256 output channels x 256 frames per tile with one accumulator in tensor memory, drained by sixteen epilogue
 * warps when the batch has at most 256 samples (else as 4); 1 = 256 x 128 and 2 = 128 x 256 with two accumulators,
 * so that a tile's epilogue overlaps the next tile's MMAs; 3 = 128 x 256, one accumulator, two CTAs per SM;
 * 4 = as 0 with eight epilogue warps; 5 = as 2 with sixteen epilogue warps (four per 32 accumulator rows; batches of
 * more than 256 samples take 2).  Other values: SC_ERR_UNSUPPORTED.  Results do not depend on the shape except
 * for the summation order of the batch-norm statistics. */
int  sepconv_set_tile_shape(sc_ctx* ctx, int shape);

/* Overlap between kernels (both forms on by default; `on` is a bit mask, 3 = both, 0 = neither).
 * Bit 0: the weight-gradient contractions of a layer and the residual projection's forward contraction do not
 * feed the next kernel of the pass; they run on a second stream that the context owns, forked from and joined
 * back into `cuda_stream` with events before the call returns.  Bit 1: every kernel is launched with
 * programmatic stream serialization: it may start (set up its barriers, allocate tensor memory) while the
 * kernel before it drains, and waits for that kernel's completion before it touches global memory.  To the
 * caller every call still behaves as work enqueued on `cuda_stream` alone (stream capture included), and the
 * results are bit-identical for every setting.  (The paper has no counterpart.) */
int  sepconv_set_overlap(sc_ctx* ctx, int on);

/* Number of kernel launches this context has enqueued so far (for reporting; the paper has no
 * counterpart). */
int64_t sepconv_launch_count(sc_ctx* ctx);

/* Per-kernel-class timing with CUDA events on the launching stream (measurement aid; the paper has
 * no counterpart).  Kernel classes are numbered 0 .. sepconv_kernel_class_count()-1 and named by
 * sepconv_kernel_class_name().  sepconv_profile_begin brackets, from now on, every launch of
 * `kernel_class` (-1: every class) with an event pair, up to max_launches launches (it creates the
 * events, host objects, on first use).  sepconv_profile_end synchronises the stream, stops the
 * bracketing and fills four HOST arrays of class-count entries: total milliseconds, number of
 * bracketed launcher calls, and the algorithmic bytes and flops those calls moved / performed
 * (padded-frame counts; every tensor read or written once). */
int  sepconv_profile_begin(sc_ctx* ctx, int kernel_class, int max_launches);
int  sepconv_profile_end(sc_ctx* ctx, void* cuda_stream, double* ms, int64_t* launches, double* bytes,
                         double* flops);
int  sepconv_kernel_class_count(void);
const char* sepconv_kernel_class_name(int kernel_class);

#ifdef __cplusplus
}
#endif
#endif /* SEPCONV_H_ */
