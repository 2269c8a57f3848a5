// Shared declarations of the H-BitLinear CUDA library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "hbl.h"

namespace hbl {

// ---- device status word (first error wins) --------------------------------
// Device address of the library's status word on the current device (host call;
// NULL if the address cannot be obtained).  Kernels receive it as a parameter.
int* device_status_word();
__device__ __forceinline__ void report_device_error(int* status, int code) { atomicCAS(status, 0, code); }

// ---- instrumentation (host side, see hbl_profile_events / hbl_launch_count) ----
enum KernelId { KERNEL_NONE = 0, KERNEL_ACT = 1, KERNEL_CONTRACT = 2, KERNEL_UNPACK = 3, KERNEL_WEIGHT = 4 };
void note_launch();                                   // +1 on the library's kernel-launch counter
void profile_before(int kernel_id, cudaStream_t s);   // records the next start event if this kernel is selected
void profile_after(int kernel_id, cudaStream_t s);

// ---- small helpers ----------------------------------------------------------
__host__ __device__ constexpr int ilog2(unsigned v) { return v <= 1 ? 0 : 1 + ilog2(v >> 1); }
inline bool is_pow2(long v) { return v > 0 && (v & (v - 1)) == 0; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Per-device state: a process may drive several GPUs, and function attributes, SM counts and symbol
// addresses belong to the device that is current when they are set or read.
constexpr int kMaxDevices = 64;
inline int current_device() {
  int dev = 0;
  return (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices) ? dev : -1;
}
int sm_count();   // multiprocessors of the current device (148 if the query fails)

#define HBL_CUDA_OK(expr)                         \
  do {                                            \
    cudaError_t _e = (expr);                      \
    if (_e != cudaSuccess) return HBL_ERR_CUDA;   \
  } while (0)

// Raises a kernel's dynamic shared-memory limit, once per device and per instantiation (the attribute is
// idempotent, so a race between host threads only repeats the call).
#define HBL_ALLOW_DYNAMIC_SMEM(kern, bytes)                                                                  \
  do {                                                                                                       \
    static bool _done[::hbl::kMaxDevices] = {};                                                              \
    const int _dev = ::hbl::current_device();                                                                \
    if (_dev < 0) return HBL_ERR_CUDA;                                                                       \
    if (!_done[_dev]) {                                                                                      \
      HBL_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(bytes)));    \
      _done[_dev] = true;                                                                                    \
    }                                                                                                        \
  } while (0)

// ---- programmatic dependent launch ----------------------------------------------
// A kernel launched with launch_dependent() may start while the kernel before it on the stream is
// still running, provided that kernel executes griddepcontrol.launch_dependents (or has exited).
// The dependent must call grid_dependency_wait() before it reads anything the earlier kernel
// writes.  The activation kernels also call it last thing, so that "kernel k has completed"
// implies "kernels before k have completed" along a chain of such launches.
//
// One kernel releases its dependents long before it ends: the streaming contraction of a call made with
// HBL_PATH_STREAM_OVERLAP.  What follows it may then run beside it, which only a call in the same mode is
// prepared for (it writes to the other half of a double-buffered workspace, and its caller has stated that its
// inputs do not come from the call before).  The library therefore remembers, per stream, whether its last
// launch was such a kernel, and gives the next launch on that stream the programmatic attribute only if that
// launch belongs to a call in the same mode; any other launch is an ordinary one and starts when everything
// before it is complete.  LaunchMode is what the entry point in charge sets for the launches it makes.
struct LaunchMode {
  bool overlap_ok = false;            // the launches of this call may run beside an early-releasing contraction
  bool releases_early = false;        // the next launch is such a contraction
};
LaunchMode& launch_mode();                                    // per host thread
bool stream_released_early(cudaStream_t s);                   // the library's last launch on s releases early
void set_stream_released_early(cudaStream_t s, bool v);
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                    Args... args) {
  const LaunchMode mode = launch_mode();
  const bool programmatic = mode.overlap_ok || !stream_released_early(s);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = programmatic ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
  set_stream_released_early(s, mode.releases_early);
  return e;
}
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- kernel launchers (one per .cu file) -------------------------------------
// Activation side: Eq. 3-6.
// packed: INT4 codes are written two per byte ([T, K / 2] bytes, layout in hbl.h) instead of one; only where
// act_quant_can_pack() says so (HBL_ERR_SHAPE otherwise), and never together with codesum or xr_out.
bool act_quant_can_pack(int x_dtype, int T, int K, int bits, int use_hadamard);
int launch_act_quant(const void* x, int x_dtype, int T, int K, int bits, int use_hadamard, float eps,
                     int8_t* codes, float* scale, int32_t* codesum, float* xr_out,
                     int32_t* zero_fill, size_t zero_fill_words, cudaStream_t s, bool packed = false);
// The same for bf16 inputs with the transform on (tensor-core first stages, packed fp32 butterflies).
bool act_quant_bf16_supported(int K);
// Several bf16 inputs of T tokens each, quantized by one launch (Eq. 3-6 per input).
constexpr int kMaxActJobs = 4;
struct ActJob { const void* x; int8_t* codes; float* scale; int32_t* codesum; int K; int use_hadamard; };
bool act_multi_bf16_supported(const ActJob* jobs, int n_jobs);
// ready (optional): n_jobs counters; every thread block adds one to its input's when its codes, scales and code
// sums are written.  blocks_out (optional): thread blocks per input.
int launch_act_multi_bf16(const ActJob* jobs, int n_jobs, int T, int bits, float eps, int32_t* zero_fill,
                          size_t zero_fill_words, cudaStream_t s, unsigned* ready = nullptr, unsigned* blocks_out = nullptr);
int launch_act_quant_bf16(const void* x, int T, int K, int bits, float eps, int8_t* codes, float* scale,
                          int32_t* codesum, float* xr_out, int32_t* zero_fill, size_t zero_fill_words,
                          cudaStream_t s, bool packed = false);
// The same with the token RMS-normalised and multiplied by gain[K] (fp32 or bf16, device) first ("LN" of Eq. 7).
int launch_norm_act_quant_bf16(const void* x, const void* gain, int gain_dtype, float norm_eps, int T, int K, int bits,
                               float eps, int8_t* codes, float* scale, int32_t* codesum, float* xr_out,
                               int32_t* zero_fill, size_t zero_fill_words, cudaStream_t s, bool packed = false);
// The same with the token replaced by SiLU(gate) * up first (both bf16 [T, K]): the SwishGLU input of W_down.
int launch_glu_act_quant_bf16(const void* gate, const void* up, int T, int K, int bits, float eps, int8_t* codes,
                              float* scale, int32_t* codesum, float* xr_out, int32_t* zero_fill, size_t zero_fill_words,
                              cudaStream_t s, bool packed = false);
// The transform alone, bf16 in and out (Eq. 8: the backward pass applies it to the gradient); K as above.
int launch_hadamard_bf16(const void* x, int T, int K, void* out, cudaStream_t s);
// Weight side: Eq. 1-2 and the 2-bit format.
int launch_weight_quant(const void* W, int w_dtype, int N, int K, float eps, void* packed, float* alpha,
                        void* ws, cudaStream_t s);
int launch_unpack_weights(const void* packed, int N, int K, int8_t* out, cudaStream_t s);
// Low-bit attention states (section 3.1): absmax quantizer at 3, 4 or 8 bits per head of each token, unsigned codes.
int launch_kv_quant(const void* x, long n_rows, int n_heads, int head_dim, int bits, int seq_len, float eps, void* codes,
                    float* scale, void* bos_codes, float* bos_scale, cudaStream_t s);
// Contraction + epilogue.  Exactly one of y / acc_out is written.
struct GemmSegment {          // one weight tensor of a (possibly fused) projection
  const void* W;              // packed (stream path) or int8 row-major (tensor path)
  const float* alpha;         // device, one float (ignored when acc_out is set)
  void* y;                    // bf16 [T, N]
  int N;
};
// early_release_reserve >= 0 (calls in HBL_PATH_STREAM_OVERLAP): the kernel releases its programmatic dependents as
// soon as it has seen the kernel before it complete, and leaves that many SMs without a thread block of its own
// for the next call's quantizer to run on; -1: neither.
// ready (same mode, optional): counters the quantizer's thread blocks raise per input when their codes are written
// (target[m] thread blocks for input m); the contraction then starts on an input's codes as soon as they are all
// there instead of when the quantizer has completed, and its last thread block clears the counters and `done`.
struct StreamReady { unsigned* ready; unsigned target[4]; unsigned* done; };
int launch_gemm_stream(const int8_t* codes, const float* scale, const int32_t* codesum, int T, int K,
                       const void* W_packed, int N, const float* alpha, __nv_bfloat16* y,
                       int32_t* acc_out, int32_t* acc_ws, int* counters, cudaStream_t s, int early_release_reserve = -1,
                       const StreamReady* ready = nullptr);
// Several weight tensors that read the same quantized input (q | k | v, up | gate), contracted as ONE matrix of
// concatenated weight rows: output i takes the rows [begin[i], begin[i] + width[i]) of W_i8, has its own alpha
// and its own bf16 tensor [T, width[i]].  begin[0] = 0, the widths of all but the last are multiples of 256.
constexpr int kMaxTensorOutputs = 3;
struct TensorOutputs {
  int n;
  int begin[kMaxTensorOutputs], width[kMaxTensorOutputs];
  __nv_bfloat16* y[kMaxTensorOutputs];
  const float* alpha[kMaxTensorOutputs];
};
int launch_gemm_tensor_multi(const void* codes, bool codes_packed, const float* scale, int T, int K, const int8_t* W_i8,
                             const TensorOutputs& outs, int32_t* acc_out, cudaStream_t s);
// codes: int8 [T, K], or (codes_packed) INT4 codes two per byte [T, K / 2] in the layout hbl.h gives.
int launch_gemm_tensor(const void* codes, bool codes_packed, const float* scale, int T, int K, const int8_t* W_i8, int N,
                       const float* alpha, __nv_bfloat16* y, int32_t* acc_out, cudaStream_t s);
// Several weight tensors, each reading one of up to four quantized inputs, per launch; one launch per 128 tokens.
int gemm_stream_max_tokens();
struct StreamInput { const int8_t* codes; const float* scale; const int32_t* codesum; int K; };
struct StreamJob { const void* W_packed; const float* alpha; __nv_bfloat16* y; int32_t* acc_out; int N; int input; };
int launch_gemm_stream_multi(const StreamInput* inputs, int n_inputs, const StreamJob* jobs, int n_jobs, int T,
                             int32_t* part, int* flags, cudaStream_t s, int early_release_reserve = -1,
                             const StreamReady* ready = nullptr);
size_t gemm_stream_acc_words(int T, int N);       // int32 words of split-K scratch (0 if none)
size_t gemm_stream_counter_words(int N);

}  // namespace hbl
