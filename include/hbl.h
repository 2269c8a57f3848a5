/* hbl.h -- C ABI of the H-BitLinear forward pass for NVIDIA B200 (sm_100a).
 *
 * The layer (BitNet v2, section 2.1, Eq. 1-7), for T tokens x[T,K] and latent
 * weights W[N,K] (row-major, K = in_dim, N = out_dim):
 *
 *   alpha = mean|W|,  W_t = RoundClip(W/(alpha+eps), -1, 1)             (Eq. 1-2)
 *   x_r   = H_m x   (orthonormal Sylvester-Hadamard, K = 2^m)            (Eq. 3-4)
 *   INT8: gamma = max|x_r|,  q = RoundClip(127/(gamma+eps) x_r, -128, 127), s = gamma/127   (Eq. 5)
 *   INT4: beta  = mean|x_r|, q = RoundClip(sqrt(7)/(beta+eps) x_r, -8, 7),   s = beta/sqrt(7) (Eq. 6)
 *   y[t,o] = alpha * s_t * sum_k W_t[o,k] q[t,k]   -> bf16                (Eq. 7)
 *
 * round() is round-half-to-even.  eps is an explicit argument (> 0).
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller, unless a
 *     parameter is documented as a host pointer.  The library allocates no
 *     device memory and frees none; scratch space is the caller's `workspace`.
 *   - Work is enqueued on the caller's stream (a cudaStream_t passed as void*;
 *     NULL is the default stream).  No entry point synchronises except
 *     hbl_check_status.
 *   - Every call returns an hbl_status_t.  Argument errors are found on the
 *     host before anything is launched.  A device-side wait that runs out
 *     records HBL_ERR_TIMEOUT in a status word that hbl_check_status reads.
 *   - Alignment: all buffers 16 bytes; workspace 1024 bytes.
 *   - Shapes: in_dim % 128 == 0, out_dim % 16 == 0, in_dim <= 32768,
 *     tokens >= 0 (0 is a no-op that returns HBL_OK).
 */
#ifndef HBL_H_
#define HBL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  HBL_OK = 0,
  HBL_ERR_NULL = 1,        /* a required pointer is NULL */
  HBL_ERR_SHAPE = 2,       /* a dimension is negative, zero where not allowed, or not a supported multiple */
  HBL_ERR_NOT_POW2 = 3,    /* use_hadamard with in_dim not a power of two (Eq. 4 needs n = 2^m) */
  HBL_ERR_BITS = 4,        /* bits not 4 or 8 (hbl_quantize_kv: not 3, 4 or 8) */
  HBL_ERR_ALIGN = 5,       /* a pointer is not aligned as required */
  HBL_ERR_WORKSPACE = 6,   /* workspace smaller than hbl_workspace_bytes() says */
  HBL_ERR_EPS = 7,         /* eps <= 0 or not finite */
  HBL_ERR_CUDA = 8,        /* a CUDA runtime / driver call failed (launch error, no device) */
  HBL_ERR_TIMEOUT = 9,     /* a bounded device-side wait expired */
  HBL_ERR_FORMAT = 10,     /* unknown dtype / path id */
  HBL_ERR_TOO_LARGE = 11   /* size beyond a stated maximum */
} hbl_status_t;

typedef enum { HBL_F32 = 0, HBL_BF16 = 1 } hbl_dtype_t;

/* Which contraction kernel hbl_forward / hbl_gemm_i32 use. */
typedef enum {
  HBL_PATH_AUTO = 0,       /* by token count.  Where that gives the streaming kernel, hbl_forward and hbl_block_forward
                              run the call in the back-to-back mode described under HBL_PATH_STREAM_OVERLAP whenever the
                              library can see for itself that the statement that mode needs holds: its last launch on the
                              stream either does not release early, or writes none of the bytes this call reads as
                              inputs, and does not use this call's workspace unless it is the very same one, base
                              and size (address ranges of its outputs and its workspace are compared with this call's
                              inputs and workspace).  Otherwise the call is launched as ordinary kernels, as HBL_PATH_STREAM always is. */
  HBL_PATH_STREAM = 1,     /* weight-streaming kernel (packed weights expanded in registers into tensor memory); tokens <= 512 */
  HBL_PATH_TENSOR = 2,     /* tcgen05 kind::i8 kernel, int32 accumulators in tensor memory */
  HBL_PATH_TENSOR_PACKED = 3, /* the same with the INT4 codes kept two per byte between the activation kernel and the
                              contraction, which widens them on the fly (bits = 4, bf16 x; HBL_ERR_SHAPE where the
                              activation kernel of the call cannot pack).  Same results, half the code traffic;
                              measured slower than HBL_PATH_TENSOR, so HBL_PATH_AUTO never picks it */
  HBL_PATH_STREAM_OVERLAP = 4 /* HBL_PATH_STREAM for calls issued back to back on one stream with no other work between
                              them (hbl_forward and hbl_block_forward): the contraction releases its programmatic
                              dependents as soon as it has seen its quantizer complete, so the next such call's
                              quantizer runs beside it and the next contraction takes over the SMs as this one's
                              thread blocks leave.  By this value the caller states (HBL_PATH_AUTO checks) that NONE OF THE CALL'S INPUTS
                              IS WRITTEN BY THE LIBRARY CALL ISSUED JUST BEFORE IT ON THE SAME STREAM (they may be
                              read while that call still runs); outputs and workspace are ordered as always.  Calls
                              on one workspace alternate between two halves of the quantizer's scratch (the
                              workspace sizes include both); with bf16 inputs the contraction starts on an input's
                              codes as soon as all thread blocks of the quantizer have counted themselves in for it
                              (counters in device memory of the library, 256 workspaces remembered per process).  Any other library call that follows on the stream is
                              launched as an ordinary kernel and waits for everything before it; a kernel of the
                              caller's own that is launched with the programmatic-serialization attribute directly
                              after such a call may start before the call has completed, as after any kernel that
                              releases its dependents, and has to wait (griddepcontrol.wait) before it reads the
                              call's outputs.  The paper has no counterpart: this is a launch configuration for
                              back-to-back latency. */
} hbl_path_t;

const char* hbl_status_string(int status);

/* Bytes of the packed ternary weight tensor for W[out_dim, in_dim]: 2 bits per
 * weight, stored as u = w + 1 in {0,1,2}, rows padded with zeros to a multiple of
 * 128: ceil(out_dim/128)*128*in_dim/4 bytes.  Layout: tiles of 128 rows x 128
 * columns, 4096 bytes each, ordered [row block][column block]; a tile is
 * [h = 0,1][row 0..127][four 32-bit words]; word v of (h, row) holds the weights
 * of row 128*rb + row in columns 128*kb + 16*(4h+v) + 4*i + b (i, b = 0..3) at
 * bit position 8*b + 2*i.  Returns 0 on bad shapes. */
size_t hbl_packed_weight_bytes(int out_dim, int in_dim);

/* Scratch bytes hbl_forward needs for up to max_tokens tokens (any bits, any path). */
size_t hbl_workspace_bytes(int max_tokens, int in_dim, int out_dim);

/* Scratch bytes hbl_quantize_weights needs. */
size_t hbl_quantize_weights_workspace_bytes(int out_dim, int in_dim);

/* Eq. 1-2.  W_latent: [out_dim, in_dim] row-major, fp32 or bf16.  Writes the
 * packed ternary tensor (hbl_packed_weight_bytes) and the fp32 alpha (device,
 * one float).  alpha is the fp64-accumulated mean rounded once to fp32; the
 * ternary decision is that of rint(W / (alpha + eps)) in IEEE fp32 with ties to
 * even, clipped to [-1, 1] -- taken as |W| > (alpha + eps) / 2, which is the same
 * decision for every fp32 (bf16) W.  A NaN weight becomes -1.  The tensor is read
 * twice (absmean, then ternarise and pack); nothing else of its size is touched. */
int hbl_quantize_weights(const void* W_latent, int w_dtype, int out_dim, int in_dim, float eps,
                         void* W_packed, float* alpha, void* workspace, size_t workspace_bytes,
                         void* stream);

/* The "weight and activation rotation" variant of the ablation (section 4.2, Table 5): the transform is
 * applied to the weights as well, W' = W H_m, and W' is ternarised in place of W; with use_hadamard = 1
 * the layer then computes Q_w(W H) Q(H x), and (W H)(H x) = W x before quantization.  The paper gives no
 * formula beyond that sentence; here each weight row is transformed (orthonormal, natural order, fp32,
 * H_m is symmetric) and Eq. 1-2 are applied to the fp32 result.  in_dim must be a power of two.
 * Workspace: hbl_quantize_weights_rotated_workspace_bytes (it holds the fp32 copy of W H), 256-byte
 * aligned.  Everything else as hbl_quantize_weights; the result equals hbl_hadamard_f32 on the rows
 * followed by hbl_quantize_weights. */
size_t hbl_quantize_weights_rotated_workspace_bytes(int out_dim, int in_dim);
int hbl_quantize_weights_rotated(const void* W_latent, int w_dtype, int out_dim, int in_dim, float eps,
                                 void* W_packed, float* alpha, void* workspace, size_t workspace_bytes,
                                 void* stream);

/* Eq. 3-7: the layer's forward pass for `tokens` tokens.
 *   x         [tokens, in_dim] fp32 or bf16
 *   W_packed  from hbl_quantize_weights;  alpha: device pointer to its scale
 *   bits      4 (Eq. 6) or 8 (Eq. 5);  use_hadamard: 1 applies Eq. 3-4 first
 *   y         [tokens, out_dim] bf16 (written)
 *   path      an hbl_path_t
 * The intermediate codes never leave the workspace (on the large-batch path INT4 codes are kept two per byte
 * there, see hbl_quantize_act_int4_packed, and widened inside the contraction).  On the large-batch path the
 * packed weights are expanded to int8 (into the workspace) on a side stream of the
 * library's, which forks from `stream` at the start of the call and joins it again
 * before the contraction: in `stream`'s order the call is complete when y is.  The
 * side stream is created by the first such call on a device (hbl_block_forward
 * shares it), so that call should come before any stream capture.  The side stream
 * and its events are one set per device: issue large-batch calls for one device from
 * one host thread at a time. */
int hbl_forward(const void* x, int x_dtype, int tokens, int in_dim,
                const void* W_packed, const float* alpha, int out_dim,
                int bits, int use_hadamard, float eps, void* y,
                void* workspace, size_t workspace_bytes, int path, void* stream);

/* hbl_forward with the normalisation of Eq. 7 ("X_r = Hadamard(LN(X))") fused in front of the transform.
 * The paper does not spell LN out; section 2 builds the model from RMS normalisation without biases, so
 * LN is taken as  x' = x / sqrt(mean_k x^2 + norm_eps) * gain[k],  computed in fp32 and rounded once to
 * bf16 (the type activations are handed on in), and x' is what Eq. 3-7 then see.
 *   x         device, bf16 [tokens, in_dim];  in_dim 2048, 4096, 8192 or 16384 (HBL_ERR_SHAPE otherwise)
 *   gain      device, [in_dim], fp32 or bf16 as gain_dtype says (HBL_F32 / HBL_BF16), 16-byte aligned,
 *             caller-owned; a bf16 gain halves what every token re-reads from L2 and is the faster of the two
 *   norm_eps  >= 0 (HBL_ERR_EPS otherwise); the transform is always on
 * Everything else as hbl_forward. */
int hbl_forward_norm(const void* x, const void* gain, int gain_dtype, float norm_eps, int tokens, int in_dim,
                     const void* W_packed, const float* alpha, int out_dim, int bits, float eps, void* y,
                     void* workspace, size_t workspace_bytes, int path, void* stream);

/* The down projection of a SwishGLU feed-forward block (section 2 lists SwishGLU among the model's
 * components and makes W_down an H-BitLinear layer) with the gating product fused in front of the
 * transform: the layer's input is  x' = SiLU(gate) * up,  SiLU(z) = z / (1 + exp(-z)), computed in fp32
 * and rounded once to bf16, so the [tokens, in_dim] product never goes to memory.
 *   gate, up  device, bf16 [tokens, in_dim], 16-byte aligned (the outputs of W_gate and W_up);
 *             in_dim 2048, 4096, 8192 or 16384 (HBL_ERR_SHAPE otherwise); the transform is always on
 * Everything else as hbl_forward.  The paper does not say which projection passes through SiLU; here it
 * is the first argument. */
int hbl_forward_glu(const void* gate, const void* up, int tokens, int in_dim, const void* W_packed,
                    const float* alpha, int out_dim, int bits, float eps, void* y, void* workspace,
                    size_t workspace_bytes, int path, void* stream);

/* The seven projections of a LLaMA-like decoder block (section 2): q, k, v and
 * up, gate are plain BitLinear layers (no transform) that share one quantized
 * input each; o and down are H-BitLinear layers (Hadamard on).  Every input is
 * supplied by the caller; attention, RoPE, SwishGLU and residuals are not part
 * of this call.  alpha7: device array of the seven per-tensor alphas in the
 * order q, k, v, o, up, gate, down.
 * x_down_in may be NULL: the feed-forward block is then chained inside the call, the down projection
 * taking SiLU(ygate) * yup (as hbl_forward_glu does) from the two outputs it has just written; ffn must
 * then be 2048, 4096, 8192 or 16384. */
typedef struct {
  const void *x_attn_in, *x_o_in, *x_ffn_in, *x_down_in; /* [T,H] [T,H] [T,H] [T,F] */
  const void *Wq, *Wk, *Wv, *Wo, *Wup, *Wgate, *Wdown;    /* packed ternary */
  const float* alpha7;
  void *yq, *yk, *yv, *yo, *yup, *ygate, *ydown;          /* bf16 outputs */
  int tokens, hidden, ffn, bits, x_dtype;
  float eps;
} hbl_block_t;

size_t hbl_block_workspace_bytes(int max_tokens, int hidden, int ffn);
int hbl_block_forward(const hbl_block_t* block /* host pointer */, void* workspace,
                      size_t workspace_bytes, int path, void* stream);

/* hbl_forward for callers whose tensors live in HOST memory (pinned for the copies
 * to be asynchronous): copies x_host -> x_stage, runs the layer, copies y_stage ->
 * y_host, all enqueued on `stream`.  x_stage / y_stage are DEVICE staging buffers
 * of tokens*in_dim*sizeof(x) and tokens*out_dim*2 bytes owned by the caller.
 * Calls of more than 2048 tokens run as a pipeline over chunks of tokens (rows are
 * independent): one chunk is copied in, one computed, one copied out at a time, on
 * the caller's stream and two side streams that the library creates on its first
 * such call on a device (so that first call should come before any stream capture).
 * In the caller's stream order the call is complete when y_host is; workspace as
 * for hbl_forward with max_tokens = tokens.  Results are those of hbl_forward.
 * No counterpart in the paper beyond Eq. 3-7 themselves. */
int hbl_forward_host(const void* x_host /* host */, int x_dtype, int tokens, int in_dim,
                     const void* W_packed, const float* alpha, int out_dim, int bits, int use_hadamard,
                     float eps, void* y_host /* host */, void* x_stage, void* y_stage,
                     void* workspace, size_t workspace_bytes, int path, void* stream);

/* Instrumentation (host-side state, not thread-safe).
 * hbl_launch_count: kernels this library has launched since it was loaded.
 * hbl_profile_events: start_events / stop_events are HOST arrays of n cudaEvent_t
 * handles owned by the caller; from now on the i-th launch of kernel class `kernel`
 * (1 = activation transform+quantize of Eq. 3-6, 2 = contraction+rescale of Eq. 7,
 * 3 = weight unpack, 4 unused) is bracketed by cudaEventRecord(start[i]) /
 * cudaEventRecord(stop[i]) on the launch's stream, until n pairs are used.
 * Each class has a slot of its own, so several can be bracketed during the same
 * calls; n = 0 switches the class off, kernel = 0 all of them.  Returns the number
 * of pairs the replaced slot (kernel = 0: all slots) had used, or -status on an
 * argument error. */
unsigned long long hbl_launch_count(void);
int hbl_profile_events(void** start_events, void** stop_events, int n, int kernel);

/* Synchronises `stream`, returns the first device-side error recorded since the
 * last call (HBL_OK if none) and clears it.  After an error it also clears the
 * counters HBL_PATH_STREAM_OVERLAP keeps in device memory of the library (the
 * quantizer's thread blocks count themselves in there; a kernel that gave up may
 * have left them mid-count). */
int hbl_check_status(void* stream);

/* Test aid (no counterpart in the paper): makes a bounded device-side wait run out on purpose.  One small
 * kernel waits, with a limit of limit_us microseconds (1 .. 1000000), on a barrier nobody ever arrives at, and
 * then leaves the way every pipelined kernel of this library leaves a wait that has run out: it records
 * HBL_ERR_TIMEOUT in the status word (hbl_check_status returns it once and clears it), raises its abort flag,
 * a second waiting role leaves because of that flag (*left_by_abort, a device int, is then set to 1), the block
 * drains, frees its tensor memory and returns.  Nothing traps or faults; the context stays usable.
 * Asynchronous on `stream`. */
int hbl_selftest_wait_timeout(int limit_us, int* left_by_abort, void* stream);

/* ---- stage-level entry points (the same kernels, exposed one step at a time) ---- */

/* Eq. 3-4 alone: xr_out[T,K] fp32 = H_m x, orthonormal, natural order. */
int hbl_hadamard_f32(const void* x, int x_dtype, int tokens, int in_dim, float* xr_out, void* stream);

/* The transform alone with bf16 in and bf16 out, for the backward pass: the gradient with respect to
 * the layer input is the same orthonormal transform applied to the gradient with respect to the
 * transformed input (section 2.2 "Training", the equation after Eq. 7; H_m is symmetric and its own
 * inverse).  out[T,K] = H_m g, natural order, fp32 arithmetic, one rounding to bf16 at the end.
 *   g, out   device, bf16 [tokens, in_dim] row-major, 16-byte aligned, caller-owned; may not alias.
 *   in_dim   2048, 4096, 8192 or 16384 (HBL_ERR_NOT_POW2 / HBL_ERR_SHAPE otherwise); tokens >= 0.
 * Asynchronous on `stream`; returns a status code, allocates nothing. */
int hbl_hadamard_bf16(const void* g, int tokens, int in_dim, void* out, void* stream);

/* The activation side of hbl_forward_glu alone: gating product, transform, quantize; xr_out as below. */
int hbl_glu_quantize_act(const void* gate, const void* up, int tokens, int in_dim, int bits, float eps,
                         int8_t* codes_out, float* scale_out, int32_t* codesum_out, float* xr_out, void* stream);

/* The activation side of hbl_forward_norm alone: normalise, transform, quantize.  With xr_out != NULL
 * nothing is quantized and xr_out[T,K] fp32 receives H_m x' instead (the other outputs may then be NULL). */
int hbl_norm_quantize_act(const void* x, const void* gain, int gain_dtype, float norm_eps, int tokens, int in_dim,
                          int bits, float eps, int8_t* codes_out, float* scale_out, int32_t* codesum_out,
                          float* xr_out, void* stream);

/* Eq. 3-6: transform (optional), per-token statistic, quantize.  codes_out: int8
 * [T,K], one code per byte; scale_out: fp32 [T] (s_t); codesum_out: int32 [T],
 * sum_k q[t,k] (may be NULL). */
int hbl_quantize_act(const void* x, int x_dtype, int tokens, int in_dim, int bits, int use_hadamard,
                     float eps, int8_t* codes_out, float* scale_out, int32_t* codesum_out, void* stream);

/* Eq. 3-4 and Eq. 6 with the quantize-AND-PACK step: INT4 codes two per byte, the form in which the large-batch
 * path of hbl_forward / hbl_block_forward keeps them (half the bytes written by the activation kernel and read
 * by the contraction, which widens them to int8 on the fly).
 *   codes_packed  device, written: [tokens, in_dim / 2] bytes, 16-byte aligned.  The 32-bit little-endian word g
 *                 of a token's row covers elements 8g .. 8g+7: byte b (0..3) of the word is
 *                 (q[8g+b] + 8) | (q[8g+b+4] + 8) << 4, with q in [-8, 7] the code of Eq. 6.  (In this order
 *                 `word & 0x0F0F0F0F` is four consecutive codes as bytes, `(word >> 4) & 0x0F0F0F0F` the next four.)
 *   scale_out     device, fp32 [tokens]
 * x must be bf16, and either use_hadamard = 1 with in_dim 2048, 4096, 8192 or 16384, or use_hadamard = 0 with
 * more than 64 tokens (HBL_ERR_SHAPE otherwise: the other activation kernels write one code per byte).
 * The codes are those of hbl_quantize_act(bits = 4), bit for bit. */
int hbl_quantize_act_int4_packed(const void* x, int x_dtype, int tokens, int in_dim, int use_hadamard, float eps,
                                 uint8_t* codes_packed, float* scale_out, void* stream);

/* Eq. 7's contraction on packed INT4 codes (layout above), on the tcgen05 kernel: acc_out[T,N] int32, exact.
 * workspace: hbl_workspace_bytes(T,K,N), 1024-byte aligned. */
int hbl_gemm_i32_int4_packed(const uint8_t* codes_packed, int tokens, int in_dim, const void* W_packed, int out_dim,
                             int32_t* acc_out, void* workspace, size_t workspace_bytes, void* stream);

/* Eq. 7's contraction alone: acc_out[T,N] int32 = sum_k W_t[o,k] * codes[t,k], exact.
 * codes: int8 [T,K].  codesum: int32 [T] (sum of each token's codes; required
 * by the streaming path, ignored by the tensor path; may be NULL with
 * HBL_PATH_TENSOR).  workspace: hbl_workspace_bytes(T,K,N). */
int hbl_gemm_i32(const int8_t* codes, const int32_t* codesum, int tokens, int in_dim,
                 const void* W_packed, int out_dim, int32_t* acc_out,
                 void* workspace, size_t workspace_bytes, int path, void* stream);

/* hbl_gemm_i32 on the streaming kernel for callers that cannot hand over a
 * workspace.  (No counterpart in the paper: this is a packaging variant of the
 * contraction above.)  Some hosts of this library may not allocate device memory
 * at the point where they call it -- an inference server that gave every spare
 * byte to its KV-cache pool at start-up, a plugin running inside a framework's
 * stream callback where an allocation would synchronise the device, a runtime
 * whose memory budget is frozen after initialisation -- and have no buffer of
 * their own to lend.  For them the kernel's scratch (partial sums handed between
 * thread blocks, and their ready flags) sits in a fixed 1.25 MiB + 4 KiB array inside
 * the library's device image; every GPU that loads the library holds it until the
 * process ends.
 *   - Inputs and the output are still the caller's: codes int8 [T,K], codesum
 *     int32 [T], W_packed, acc_out int32 [T,N], all device pointers.
 *   - Limit: tokens <= 16 (any out_dim); more tokens return HBL_ERR_TOO_LARGE before
 *     any work is enqueued.
 *   - The call allocates and frees nothing.  The first call on each device looks up
 *     the array's device address (that device must be current); make that first
 *     call outside any stream capture.
 *   - Every call reuses the same array, which keeps the previous call's contents, and
 *     clears the ready flags (the only part that must start at zero) on `stream`
 *     first.  Two calls that can overlap on the GPU (different streams, no ordering
 *     between them) race on it: order them. */
int hbl_gemm_i32_static(const int8_t* codes, const int32_t* codesum, int tokens, int in_dim,
                        const void* W_packed, int out_dim, int32_t* acc_out, void* stream);

/* Low-bit attention states (section 3.1 "Inference", Tables 2-3): the Q, K and V heads are quantized after the
 * rotary embedding "to unsigned integers using the absmax function" (4-bit, or 3-bit for the KV cache), and the
 * K/V heads of the [BOS] token are kept at 8 bits.  The paper prints no formula; the one used is Eq. 5's absmax
 * quantizer at b bits with one statistic per head of each token, stored with an offset so that it is unsigned:
 *   gamma = max_d |x[d]|,  q = RoundClip((2^(b-1) - 1) / (gamma + eps) * x, -2^(b-1), 2^(b-1) - 1),
 *   u = q + 2^(b-1) in [1, 2^b - 1],  scale = gamma / (2^(b-1) - 1),  so that  x ~ scale * (u - 2^(b-1)).
 * The decision is taken in IEEE fp32 in the order written (division, product, round-half-to-even, clip).
 *   x          device, bf16 [tokens, n_heads, head_dim] contiguous (the states after RoPE), 16-byte aligned
 *   head_dim   64, 128 or 256 (HBL_ERR_SHAPE otherwise);  bits 3, 4 or 8 (HBL_ERR_BITS otherwise);  eps > 0
 *   codes      device, written: hbl_kv_codes_bytes() bytes, 16-byte aligned.  Each head is a run of
 *              head_dim * bits / 8 bytes; element d of the head is the bits [bits * d, bits * d + bits) of that
 *              run read as a little-endian bit string (4 bits: element 2j in the low nibble of byte j)
 *   scale      device, written: fp32 [tokens * n_heads]
 *   bos_codes  device or NULL.  Not NULL: tokens t with t % seq_len == 0 (seq_len > 0: the first token of each
 *              sequence of a [n_seq, seq_len] batch) are the [BOS] tokens; their heads are quantized at 8 bits
 *              as well, into bos_codes [ceil(tokens / seq_len), n_heads, head_dim] (one byte per element) and
 *              bos_scale [ceil(tokens / seq_len) * n_heads]; a reader of the cache takes these for position 0
 * All buffers are the caller's; asynchronous on `stream`; nothing is allocated.  hbl_kv_codes_bytes returns 0
 * for an unsupported shape. */
size_t hbl_kv_codes_bytes(int tokens, int n_heads, int head_dim, int bits);
int hbl_quantize_kv(const void* x, int tokens, int n_heads, int head_dim, int bits, int seq_len, float eps, void* codes,
                    float* scale, void* bos_codes, float* bos_scale, void* stream);

/* Packed ternary -> int8 [N,K] row-major, values in {-1,0,1}. */
int hbl_unpack_weights(const void* W_packed, int out_dim, int in_dim, int8_t* w_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HBL_H_ */
