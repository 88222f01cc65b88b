/*
 * qasr.h -- C ABI of the integer-only Q-ASR encoder library (CUDA, sm_100a).
 *
 * The library runs the forward pass of QuartzNet / Jasper style 1-D convolutional
 * speech encoders entirely in integer arithmetic (arXiv 2103.16827, Sec. 2.2):
 * int8 activations, per-channel int8 weights, int32 accumulation, BatchNorm
 * folded into weights and an int32 bias, dyadic requantisation, integer ReLU and
 * integer residual adds.  The only floating-point operation is the final
 * dequantisation of the logits (Sec. 2.1, DQ(q, S) = S * q).
 *
 * Conventions common to every call
 *   - Tensors are dense, row-major [B][C][T] with time contiguous.
 *   - Every data pointer is a DEVICE pointer owned by the caller unless the
 *     comment says "host".  The library keeps no reference after the work it
 *     enqueued has finished.
 *   - Work is enqueued on the stream given to qasr_create and the call returns
 *     without waiting; inputs and outputs must stay alive until that stream has
 *     been synchronised.  In-place operation (output == an input) is rejected.
 *   - Return value: 0 on success, a negative QASR_ERR_* code otherwise.  Argument
 *     errors are detected on the host before anything is launched.  Nothing
 *     throws, aborts or traps.  qasr_last_error gives a sticky description.
 *   - Arithmetic definitions
 *       RS(v, c)  = floor((v + 2^(c-1)) / 2^c) on a signed 64-bit v, 1 <= c <= 62
 *       sat8(v)   = min(127, max(-128, v))               (the b = 8 grid of Eq. 1)
 *       requant   = sat8(RS((int64)acc * mult[ch], shift[ch])), 0 <= mult < 2^31
 *     Convolutions are cross-correlations with zero padding dilation*(K-1)/2 on
 *     both sides, K odd; T_out = (T - 1) / stride + 1.
 *   - mult/shift arrays live on the device, so their range is checked by the
 *     kernels: an out-of-range entry sets a sticky device status that
 *     qasr_poll_status reports as QASR_ERR_RANGE (the affected outputs are
 *     unspecified but every access stays in bounds).
 */
#ifndef QASR_H_
#define QASR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define QASR_OK 0
#define QASR_ERR_NULL (-1)            /* a required pointer is NULL */
#define QASR_ERR_SHAPE (-2)           /* non-positive size, even K, K > 127, stride/dilation not in {1,2}, ... */
#define QASR_ERR_ALIGN (-3)           /* an int32/float pointer is not 4-byte aligned */
#define QASR_ERR_RANGE (-4)           /* shift outside [1,62] or negative multiplier */
#define QASR_ERR_OVERFLOW_RISK (-5)   /* taps*127*128 + max|bias| >= 2^31: int32 wrap-around cannot be excluded */
#define QASR_ERR_WORKSPACE (-6)       /* workspace missing, misaligned or too small */
#define QASR_ERR_CUDA (-7)            /* a CUDA runtime/driver call failed; text in qasr_last_error */
#define QASR_ERR_DEVICE_TIMEOUT (-8)  /* a bounded device-side wait expired */
#define QASR_ERR_TABLE (-9)           /* inconsistent layer table (buffer ids, channel counts, order) */
#define QASR_ERR_ALIAS (-10)          /* output aliases an input */
#define QASR_ERR_TOO_LARGE (-11)      /* the operation needs more than the built-in static scratch holds */

#define QASR_MAX_TERMS 12

typedef struct qasr_ctx qasr_ctx; /* opaque: device, stream, status word, cached launch plans */

/* Per-channel dyadic requantisation constants: device arrays of length C. */
typedef struct qasr_requant {
    const int32_t* mult;
    const uint8_t* shift;
} qasr_requant;

/* ---- context -------------------------------------------------------------------------- */

/* Creates a context bound to `device` and to `cuda_stream` (a cudaStream_t passed as void*,
 * borrowed, may be NULL for the default stream).  Allocates a small device status word.
 * *out is set only on success. */
int qasr_create(qasr_ctx** out, int device, void* cuda_stream);

/* Waits for the context's stream, frees what qasr_create and the plan cache allocated. */
int qasr_destroy(qasr_ctx* ctx);

/* Static text for a return code; never NULL. */
const char* qasr_strerror(int code);

/* Sticky description of the last error seen by this context ("" if none). */
const char* qasr_last_error(const qasr_ctx* ctx);

/* Synchronises the context's stream and reads (and clears) the device status word.
 * Returns QASR_OK, QASR_ERR_RANGE, QASR_ERR_DEVICE_TIMEOUT or QASR_ERR_CUDA. */
int qasr_poll_status(qasr_ctx* ctx);

/* Options.  QASR_OPT_GRAPH (default 1): qasr_encoder_forward replays a captured CUDA graph when
 * called again with identical arguments.  QASR_OPT_TENSOR_CORES (default 1): pointwise/dense
 * convolutions use the tcgen05 path when the shape allows it (0 forces the generic kernels).
 * (Option id 3 is not in use.) */
#define QASR_OPT_GRAPH 1
#define QASR_OPT_TENSOR_CORES 2
/* QASR_OPT_PROFILE (default 0): every kernel is launched on its own (no graph) between two CUDA
 * events; qasr_profile_read returns one record per launch. */
#define QASR_OPT_PROFILE 4
/* QASR_OPT_STATIC_WEIGHTS (default 0): the caller promises that the weight tensors a layer table points
 * to do not change between calls of qasr_encoder_forward that repeat the same arguments; the per-tap
 * regrouped copies of K-tap weights that the first such call leaves in the workspace are then reused
 * instead of being rebuilt on every call (the workspace must then be left untouched between the calls).
 * Setting the option (to either value) forgets what is cached. */
#define QASR_OPT_STATIC_WEIGHTS 5
/* Tuning aids (default 0 = the library chooses).  QASR_OPT_GEMM_FRAME_TILE: frames per work item of the
 * pointwise tensor-core GEMM (a multiple of 16 in [16, 256]; at most 128 when C_in > 512).
 * QASR_OPT_DW_FRAME_TILE: frames per window of the tensor-core depthwise kernel (a multiple of 16 in
 * [16, 256]).  A value that does not fit the shape at hand is ignored for that call.  Results do not depend
 * on either; they exist so that the built-in choice can be checked against the alternatives. */
#define QASR_OPT_GEMM_FRAME_TILE 6
#define QASR_OPT_DW_FRAME_TILE 7
/* QASR_OPT_SIDE_BRANCH (default 1): inside the captured graph of qasr_encoder_forward a pointwise layer whose
 * output the next layer does not read (a block's residual projection) runs beside the main chain, on the SMs the
 * main chain's kernels leave idle, and is joined in front of the first layer that needs it.  Results do not depend
 * on the option. */
#define QASR_OPT_SIDE_BRANCH 8
/* QASR_OPT_FRAME_MAJOR_OUTPUT (default 1): inside qasr_encoder_forward a K-tap convolution on the tensor cores
 * whose output the next K-tap convolution of the table reads (stride 1) writes that output a second time from
 * its epilogue, frame-major, into the workspace, so that the reader needs no transpose kernel in front of it
 * (Sec. 3's Jasper blocks are runs of such layers).  Results do not depend on the option. */
#define QASR_OPT_FRAME_MAJOR_OUTPUT 9
int qasr_set_option(qasr_ctx* ctx, int option, int value);

/* One kernel launch seen in profile mode: which table layer it belongs to (-1 outside
 * qasr_encoder_forward), which kernel (qasr_kernel_name), its device time, and the work the
 * method itself requires of it: multiply-accumulates and bytes of tensors read + written. */
typedef struct qasr_profile_entry {
    int32_t layer;
    int32_t kernel;
    float ms;
    float reserved;
    double macs;
    double bytes;
} qasr_profile_entry;

/* Waits for the stream, copies up to `capacity` records (oldest first) to `out` (host), stores
 * the number of records that existed in *n and clears them. */
int qasr_profile_read(qasr_ctx* ctx, qasr_profile_entry* out, int capacity, int* n);

/* Name of a kernel id found in qasr_profile_entry.kernel; "?" if unknown. */
const char* qasr_kernel_name(int kernel);

/* Number of kernels this context has launched (graph replays count their kernel nodes). */
int64_t qasr_launch_count(const qasr_ctx* ctx);

/* Diagnostic: checks the library's own failure detection.  Every wait inside the tensor-core kernels
 * (on a TMA copy, on the tensor pipe, on a free buffer) is bounded; when one expires the kernel raises a
 * sticky status that qasr_poll_status reports as QASR_ERR_DEVICE_TIMEOUT, releases its tensor memory and
 * ends normally.  This call enqueues one tiny kernel that runs exactly that path on purpose: it sets up
 * as those kernels do, waits limit_us microseconds (1 .. 1 000 000) on a barrier that nothing signals,
 * gives up and tears down.  Afterwards qasr_poll_status returns QASR_ERR_DEVICE_TIMEOUT once, and the
 * context works as before.  (No passage of the paper: an operational aid.)  sm_100 devices only. */
int qasr_selftest_wait_timeout(qasr_ctx* ctx, unsigned limit_us);

/* Diagnostic: the int8 tensor-core throughput this GPU reaches on the instruction the convolution kernels
 * use (tcgen05.mma kind::i8, M = 128, N = 256, K = 32), issued back to back by every SM on operands that
 * stay in shared memory -- the denominator for "fraction of the int8 tensor peak".  Runs `kblocks` groups
 * of four such instructions per SM (1 .. 2^20; 20 000 take about a millisecond), waits for them, and
 * returns the device time in *ms (host pointer) and the operations done in *ops (a multiply-accumulate
 * counts as two).  Blocking.  (No passage of the paper: a measurement aid.)  sm_100 devices only. */
int qasr_measure_int8_tensor_peak(qasr_ctx* ctx, int kblocks, float* ms, double* ops);

/* ---- single operations ------------------------------------------------------------------ */

/* Depthwise K-tap convolution with per-channel requantisation (no bias, no ReLU): the
 * time-wise half of a time-channel-separable block, an integer convolution in the sense of
 * Sec. 2.2.
 *   acc[b,c,t] = sum_k w_dw[c,k] * x[b,c,t*stride + k*dilation - pad];  y = requant(acc)
 * x [B][C][T] int8, w_dw [C][K] int8, y [B][C][T_out] int8. K odd, 1 <= K <= 127. */
int qasr_dw_conv(qasr_ctx* ctx, const int8_t* x, int B, int C, int T,
                 const int8_t* w_dw, int K, int stride, int dilation, qasr_requant rq_dw,
                 int8_t* y);

/* Pointwise (K == 1) or dense K-tap convolution with folded-BatchNorm bias and the fused
 * epilogue (Sec. 2.2: integer conv, folded BN, integer ReLU):
 *   acc[b,o,t] = bias[o] + sum_i sum_k w[o,i,k] * x[b,i,t*stride + k*dilation - pad]
 *   a = requant(acc)                                        (int8, no ReLU yet)
 *   n_terms == 0:  y = relu ? max(a,0) : a
 *   n_terms >= 2:  v = RS(a*term_mult[0], term_shift[0]) + sum_{j>=1} RS(terms[j]*term_mult[j], term_shift[j])
 *                  y = sat8(relu ? max(v,0) : v)             (terms[0] is ignored)
 *   y_int32 != NULL: the raw accumulator acc is stored there instead (no requant), y unused.
 * w [C_out][C_in][K] int8, bias [C_out] int32 or NULL, max_abs_bias >= max|bias| (host value used
 * for the overflow check), terms: host array of n_terms device pointers [B][C_out][T_out],
 * term_mult/term_shift: host arrays. */
int qasr_conv(qasr_ctx* ctx, const int8_t* x, int B, int C_in, int T,
              const int8_t* w, int C_out, int K, int stride, int dilation,
              const int32_t* bias, int32_t max_abs_bias, qasr_requant rq, int relu,
              int n_terms, const int8_t* const* terms, const int32_t* term_mult,
              const uint8_t* term_shift, int8_t* y, int32_t* y_int32);

/* Scratch for the tensor-core path of qasr_conv.  A K-tap (or strided) convolution runs on the
 * tensor cores as an implicit GEMM over (input channel, tap); that path first writes a frame-major
 * copy of x and a per-tap regrouping of w into device scratch that the caller lends to the context:
 *   qasr_conv_scratch_bytes: bytes one such convolution wants (the arithmetic and its results are
 *     those of qasr_conv either way);
 *   qasr_set_conv_scratch: lends [scratch, scratch + bytes) to the context (device memory, 256-byte
 *     aligned, owned by the caller, must outlive every later qasr_conv on this context; NULL/0 takes
 *     it back).  Without scratch, or with too little, qasr_conv uses the generic kernel.
 * qasr_encoder_forward does not use this region: its own workspace already includes the scratch. */
int qasr_conv_scratch_bytes(int B, int C_in, int C_out, int T, int K, int stride, size_t* bytes);
int qasr_set_conv_scratch(qasr_ctx* ctx, void* scratch, size_t bytes);

/* One QuartzNet time-channel-separable block (Sec. 3 names the QuartzNet encoders; Sec. 2.2 defines
 * the integer-only operators it is made of: integer convolution on the quantised operands, BatchNorm
 * folded into the preceding convolution, ReLU on integers): depthwise K-tap conv + requant, then
 * pointwise 1x1 conv with folded-BN bias, requant and optional ReLU (qasr_dw_conv followed by
 * qasr_conv with K = 1, bit for bit).  x [B][C_in][T] -> y [B][C_out][T_out].
 * workspace: device scratch of at least qasr_tcs_block_workspace_bytes (may be NULL when that
 * is 0), 256-byte aligned; its contents are unspecified afterwards. */
int qasr_tcs_block_workspace_bytes(int B, int C_in, int C_out, int T, int K, int stride,
                                   int dilation, size_t* bytes);
int qasr_tcs_block(qasr_ctx* ctx, const int8_t* x, int B, int C_in, int T,
                   const int8_t* w_dw, int K, int stride, int dilation, qasr_requant rq_dw,
                   const int8_t* w_pw, int C_out, const int32_t* bias, int32_t max_abs_bias,
                   qasr_requant rq_pw, int relu, int8_t* y,
                   void* workspace, size_t workspace_bytes);

/* The same block for callers that are not allowed to allocate device memory -- for instance a
 * streaming recogniser's audio callback running under a fixed memory budget, a serving plugin
 * whose enqueue hook may not touch the allocator, or a process in which another component has
 * reserved the whole device.  (The paper has no counterpart: this is an integration aid, not a
 * step of the method.)  It needs no context and no workspace: the depthwise output is kept in a
 * static device array that is part of the library image, so every GPU that loads the library
 * holds QASR_NOALLOC_SCRATCH_BYTES until the process exits, and the call itself never allocates
 * or frees anything.
 *   - Same arithmetic and argument meaning as qasr_tcs_block; the result is bit-identical.
 *   - device / cuda_stream: where to run (cudaStream_t as void*, NULL = default stream).
 *   - Limit: B * C_in * T_out <= QASR_NOALLOC_SCRATCH_BYTES, otherwise QASR_ERR_TOO_LARGE is
 *     returned and nothing is launched.
 *   - The first call on each device looks up the array's device address and sets kernel
 *     attributes; make that first call before starting any stream capture.
 *   - Every call on a device shares the one array, which simply keeps what the last call left in
 *     it (nothing in it needs to start at zero: each call overwrites the part it reads).  Two
 *     calls whose kernels overlap on the GPU (different streams, no ordering) race on it;
 *     serialise them.
 *   - wait != 0: the call waits for the stream and also reports (and clears) the device status,
 *     i.e. QASR_ERR_RANGE for an out-of-range mult/shift entry.  wait == 0: asynchronous.
 *   - Besides the array, all calls on a device share ONE status word, and it is sticky: an error
 *     that a wait == 0 call leaves there is neither reported nor cleared until some later call
 *     with wait != 0 on that device collects it -- possibly another caller's, on another stream
 *     (and clearing it races with kernels of other streams still in flight).  Callers that run
 *     asynchronously should therefore finish each batch of calls with one wait != 0 call.
 *   - wait != 0 synchronises the stream and copies the status word back with a blocking copy, so
 *     it cannot be used while the stream is being captured, not even after the first call.
 *   - The call makes `device` the calling thread's current CUDA device and leaves it so. */
#define QASR_NOALLOC_SCRATCH_BYTES (16u << 20)
int qasr_tcs_block_noalloc(int device, void* cuda_stream,
                           const int8_t* x, int B, int C_in, int T,
                           const int8_t* w_dw, int K, int stride, int dilation, qasr_requant rq_dw,
                           const int8_t* w_pw, int C_out, const int32_t* bias, int32_t max_abs_bias,
                           qasr_requant rq_pw, int relu, int8_t* y, int wait);

/* Integer residual add of int8 tensors that sit at different scales (Sec. 2.2 requires the entire
 * inference, the residual connections of the encoders included, to run in integer arithmetic; it does
 * not print the rule, so the per-term dyadic rescaling below is this library's reading of it):
 *   y = sat8(relu?( sum_j RS(terms[j] * mult[j], shift[j]) )),  every term rounded on its own.
 * terms: host array of n_terms (1..QASR_MAX_TERMS) device pointers [B][C][T]; mult, shift: host
 * arrays (per-tensor constants). */
int qasr_residual_requant_add(qasr_ctx* ctx, int n_terms, const int8_t* const* terms,
                              const int32_t* mult, const uint8_t* shift,
                              int B, int C, int T, int relu, int8_t* y);

/* Integer gated linear unit of the Conformer convolution module.  Sec. 2.2 says the non-linearities
 * are replaced by 2nd-order polynomials on integers but prints no coefficients, so the gate below is
 * this library's own definition (a piecewise-quadratic sigmoid that saturates at |g| = q_c):
 *   x [B][2C][T] int8: a = channels [0, C), g = channels [C, 2C)
 *   u = min(|g|, q_c);  p = q_c - u;  h = 2 q_c^2 - p^2;  sig = g >= 0 ? h : 2 q_c^2 - h
 *   y[b,c,t] = sat8(RS(a * sig * mult[c], shift[c]))                y [B][C][T] int8
 * 1 <= q_c <= 128. */
int qasr_glu(qasr_ctx* ctx, const int8_t* x, int B, int C, int T, int q_c, qasr_requant rq, int8_t* y);

/* Final dequantisation (Sec. 2.1, DQ): out[b,c,t] = (float)acc[b,c,t] * scale[c], one IEEE
 * fp32 multiply per element. scale: device array [C]. */
int qasr_dequant_logits(qasr_ctx* ctx, const int32_t* acc, int B, int C, int T,
                        const float* scale, float* out);

/* ---- whole encoder ---------------------------------------------------------------------- */

#define QASR_LAYER_DW 1     /* qasr_dw_conv */
#define QASR_LAYER_PW 2     /* qasr_conv with K = 1 */
#define QASR_LAYER_DENSE 3  /* qasr_conv with K taps */
#define QASR_LAYER_TCS 4    /* qasr_tcs_block (+ optional residual terms on the pointwise output) */
#define QASR_LAYER_ADD 5    /* qasr_residual_requant_add over term_buf[0..n_terms) */
#define QASR_LAYER_GLU 6    /* qasr_glu: C_in = 2 * C_out channels in, C_out out, constants in rq, glu_qc */

/* One entry of the layer table (host memory, plain data).  Activation buffers are named by
 * small integers: 0 is the encoder input, ids >= 1 live in the caller's workspace; a buffer may
 * be written by several layers (ping-pong), its size is the largest tensor written to it.  A
 * layer with out_int32 != 0 must be the last one; it writes the int32 logits. */
typedef struct qasr_layer {
    int32_t kind;
    int32_t in_buf;
    int32_t out_buf;
    int32_t C_in, C_out;
    int32_t K, stride, dilation;
    const int8_t* w_dw;   /* [C_in][K]            (DW, TCS) */
    qasr_requant rq_dw;   /* [C_in]               (DW, TCS) */
    const int8_t* w;      /* [C_out][C_in][K]     (PW, DENSE, TCS: K = 1) */
    const int32_t* bias;  /* [C_out] or NULL */
    int32_t max_abs_bias;
    qasr_requant rq;      /* [C_out] */
    int32_t relu;
    int32_t out_int32;
    int32_t glu_qc;                        /* GLU only: the gate saturates at |g| = glu_qc */
    int32_t n_terms;                       /* 0, or 1 + number of residual buffers (ADD: number of terms) */
    int32_t term_buf[QASR_MAX_TERMS];      /* term_buf[0] is ignored unless kind == ADD */
    int32_t term_mult[QASR_MAX_TERMS];
    uint8_t term_shift[QASR_MAX_TERMS];
} qasr_layer;

/* sizeof(qasr_layer) as the library was compiled, for bindings that mirror the struct. */
size_t qasr_layer_size(void);

/* Bytes of device workspace qasr_encoder_forward needs for this table at batch B, length T
 * (activation buffers plus internal scratch).  Validates the table. */
int qasr_encoder_workspace_bytes(const qasr_layer* table, int n_layers, int B, int C_in, int T,
                                 size_t* bytes);

/* Forward pass over a layer table (the encoders of Sec. 3 as data): x [B][C_in][T] int8 ->
 * logits_q [B][C_last][T_last] int32 (the last layer's accumulator + bias) and, if logits and
 * out_scale are non-NULL, logits = DQ(logits_q, out_scale).  The table is validated completely
 * before anything is launched.  workspace must be 256-byte aligned. */
int qasr_encoder_forward(qasr_ctx* ctx, const qasr_layer* table, int n_layers,
                         const int8_t* x, int B, int C_in, int T,
                         void* workspace, size_t workspace_bytes,
                         int32_t* logits_q, float* logits, const float* out_scale);

/* Where buffer `buf_id` of the table lives inside the workspace (for inspecting intermediate
 * tensors): byte offset and shape [B][*C][*T_len]. */
int qasr_encoder_buffer_info(const qasr_layer* table, int n_layers, int B, int C_in, int T,
                             int buf_id, size_t* offset, int* C, int* T_len);

/* Host variant for callers whose data lives in host memory: copies x to the device, runs
 * qasr_encoder_forward, copies logits_q/logits back and waits.  x, logits_q and logits are HOST
 * pointers (pinned memory makes the copies asynchronous); table constants, workspace and
 * out_scale are device pointers as above; staging is carved from the end of the workspace, so
 * workspace_bytes must be at least qasr_encoder_workspace_bytes + qasr_encoder_host_staging_bytes. */
int qasr_encoder_host_staging_bytes(const qasr_layer* table, int n_layers, int B, int C_in, int T,
                                    size_t* bytes);
int qasr_encoder_forward_host(qasr_ctx* ctx, const qasr_layer* table, int n_layers,
                              const int8_t* x_host, int B, int C_in, int T,
                              void* workspace, size_t workspace_bytes,
                              int32_t* logits_q_host, float* logits_host, const float* out_scale);

/* Pipelined host variant for callers that stream batch after batch (Sec. 3.2 deploys the encoder as a whole-model
 * forward per call): qasr_encoder_forward_host_async only enqueues -- input copy, forward pass, result copies --
 * and returns; the copies run on streams of the context's own, so that with two slots used in turn the copies of
 * one call overlap the kernels of the other.  qasr_encoder_host_wait(slot) blocks until the results of the last
 * call on that slot are in host memory (and returns at once if there is none).
 *   - slot is 0 or 1; each has its own device staging, carved from the end of the workspace, so workspace_bytes
 *     must be at least qasr_encoder_host_pipeline_bytes.  A call on a slot first waits (on the host) for that
 *     slot's previous results.
 *   - x_host, logits_q_host, logits_host: HOST pointers (pinned memory, else the copies are not asynchronous); they
 *     must stay valid, and x_host unchanged, until qasr_encoder_host_wait(slot) has returned.
 *   - The kernels run on the context's stream in call order; device errors surface through qasr_poll_status.
 *   - Not usable while the context's stream is being captured. */
int qasr_encoder_host_pipeline_bytes(const qasr_layer* table, int n_layers, int B, int C_in, int T, size_t* bytes);
int qasr_encoder_forward_host_async(qasr_ctx* ctx, const qasr_layer* table, int n_layers,
                                    const int8_t* x_host, int B, int C_in, int T,
                                    void* workspace, size_t workspace_bytes,
                                    int32_t* logits_q_host, float* logits_host, const float* out_scale, int slot);
int qasr_encoder_host_wait(qasr_ctx* ctx, int slot);

#ifdef __cplusplus
}
#endif
#endif /* QASR_H_ */
