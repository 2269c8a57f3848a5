// extern "C" entry points of the H-BitLinear library: argument validation,
// workspace carving and kernel dispatch.  No device memory is allocated here.
#include <math.h>

#include <mutex>

#include "hbl_common.cuh"

using namespace hbl;

namespace hbl {
namespace {
__device__ int g_status = 0;
}
int* device_status_word() {
  // One address per device; looked up once per device (a process may use several).
  static int* cached[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (cached[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_status) != cudaSuccess) return nullptr;
    cached[dev] = static_cast<int*>(p);
  }
  return cached[dev];
}

int sm_count() {
  static int cached[kMaxDevices] = {};
  const int dev = current_device();
  if (dev < 0) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

// ---- host-side memory of early-releasing launches (see launch_dependent) ----
namespace {
std::mutex g_overlap_mutex;
constexpr int kStreamSlots = 64, kWorkspaceSlots = 256;
constexpr int kMaxRecordedOutputs = 8;
struct ByteRange { const char* lo; const char* hi; };
struct StreamSlot {
  cudaStream_t s; bool used, early;
  int n_out; ByteRange out[kMaxRecordedOutputs];             // what the early-releasing call writes (its outputs)
} g_streams[kStreamSlots] = {};
bool g_stream_overflow = false;       // an early release on a stream that found no slot: every unknown stream counts as early
struct WorkspaceSlot { const void* ws; bool used; int last; } g_workspaces[kWorkspaceSlots] = {};
}
LaunchMode& launch_mode() {
  static thread_local LaunchMode mode;
  return mode;
}
bool stream_released_early(cudaStream_t s) {
  std::lock_guard<std::mutex> lock(g_overlap_mutex);
  for (int i = 0; i < kStreamSlots; ++i)
    if (g_streams[i].used && g_streams[i].s == s) return g_streams[i].early;
  return g_stream_overflow;
}
void set_stream_released_early(cudaStream_t s, bool v) {
  std::lock_guard<std::mutex> lock(g_overlap_mutex);
  int free_slot = -1;
  for (int i = 0; i < kStreamSlots; ++i) {
    if (g_streams[i].used && g_streams[i].s == s) { g_streams[i].early = v; return; }
    if (!g_streams[i].used && free_slot < 0) free_slot = i;
  }
  if (!v && !g_stream_overflow) return;                       // nothing to remember
  if (free_slot >= 0) { g_streams[free_slot] = {}; g_streams[free_slot].s = s; g_streams[free_slot].used = true; g_streams[free_slot].early = v; }
  else if (v) g_stream_overflow = true;
}
namespace {
// The outputs of the early-releasing call just launched on s (called right after set_stream_released_early(s, true)).
void record_stream_outputs(cudaStream_t s, const ByteRange* out, int n) {
  std::lock_guard<std::mutex> lock(g_overlap_mutex);
  for (int i = 0; i < kStreamSlots; ++i)
    if (g_streams[i].used && g_streams[i].s == s) {
      g_streams[i].n_out = n < kMaxRecordedOutputs ? n : kMaxRecordedOutputs;
      for (int k = 0; k < g_streams[i].n_out; ++k) g_streams[i].out[k] = out[k];
      if (n > kMaxRecordedOutputs) g_streams[i].n_out = -1;   // unknown extent: everything may be written
      return;
    }
}
// May a quantizer that reads `in` and writes into the workspace `ws` run beside the library's last launch on s?
// Yes if that launch does not release its dependents early (the quantizer then starts after it anyway), or if it
// writes none of the bytes read and touches none of the workspace -- except that the very same workspace (same
// base, same size: same layout) is fine, its two halves taking turns.
bool clear_of_last_call(cudaStream_t s, const ByteRange* in, int n, const ByteRange& ws) {
  std::lock_guard<std::mutex> lock(g_overlap_mutex);
  for (int i = 0; i < kStreamSlots; ++i)
    if (g_streams[i].used && g_streams[i].s == s) {
      if (!g_streams[i].early) return true;
      if (g_streams[i].n_out < 0) return false;
      for (int k = 0; k < g_streams[i].n_out; ++k) {
        const ByteRange& o = g_streams[i].out[k];
        for (int j = 0; j < n; ++j)
          if (in[j].lo < o.hi && o.lo < in[j].hi) return false;
        if (ws.lo < o.hi && o.lo < ws.hi && !(ws.lo == o.lo && ws.hi == o.hi)) return false;
      }
      return true;
    }
  return !g_stream_overflow;
}
ByteRange byte_range(const void* p, size_t bytes) { return {static_cast<const char*>(p), static_cast<const char*>(p) + bytes}; }
}  // namespace
namespace {
// Which half of the double-buffered activation scratch the next overlapping call on this workspace writes:
// the one the call before it did not (0, 1, 0, ...); -1 when the table is full (the call then runs unoverlapped).
int next_overlap_half(const void* ws, int* slot) {
  std::lock_guard<std::mutex> lock(g_overlap_mutex);
  int free_slot = -1;
  for (int i = 0; i < kWorkspaceSlots; ++i) {
    if (g_workspaces[i].used && g_workspaces[i].ws == ws) { g_workspaces[i].last ^= 1; *slot = i; return g_workspaces[i].last; }
    if (!g_workspaces[i].used && free_slot < 0) free_slot = i;
  }
  if (free_slot < 0) return -1;
  g_workspaces[free_slot] = {ws, true, 0};
  *slot = free_slot;
  return 0;
}
// Counters of the back-to-back mode, per remembered workspace and half: [0..3] thread blocks of the quantizer that
// have written input m's codes, [4] thread blocks of the contraction that are through.  Zero when the module is
// loaded; the contraction's last thread block puts them back to zero, so they are zero whenever a call starts.
__device__ unsigned g_overlap_counters[kWorkspaceSlots][2][8];
unsigned* overlap_counters(int slot, int half) {
  static unsigned* base[kMaxDevices] = {};
  const int dev = current_device();
  if (dev < 0) return nullptr;
  if (base[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_overlap_counters) != cudaSuccess) return nullptr;
    base[dev] = static_cast<unsigned*>(p);
  }
  return base[dev] + ((size_t)slot * 2 + half) * 8;
}
}  // namespace

namespace {
unsigned long long g_launches = 0;
// One slot per kernel class, so that several classes can be bracketed during the same calls.
struct Profile { void** starts = nullptr; void** stops = nullptr; int n = 0, next = 0; bool open = false; } g_prof[KERNEL_WEIGHT + 1];
}
void note_launch() { ++g_launches; }
void profile_before(int kernel_id, cudaStream_t s) {
  Profile& pr = g_prof[kernel_id];
  if (pr.next >= pr.n) return;
  cudaEventRecord(static_cast<cudaEvent_t>(pr.starts[pr.next]), s);
  pr.open = true;
}
void profile_after(int kernel_id, cudaStream_t s) {
  Profile& pr = g_prof[kernel_id];
  if (!pr.open) return;
  cudaEventRecord(static_cast<cudaEvent_t>(pr.stops[pr.next]), s);
  pr.open = false;
  ++pr.next;
}
}  // namespace hbl

namespace {

constexpr int kFuseMaxTokens = 2048;      // decoder block, large batch: q|k|v and up|gate as one contraction each up to here
constexpr int kStreamMaxTokens = 512;     // = gemm_stream_max_tokens(): four passes of 128 token columns
constexpr int kMaxInDim = 32768;

struct ForwardWs {           // byte offsets inside the caller's workspace
  size_t scale, codesum, zero_region, counters, acc, codes, w_i8, total;
  size_t zero_words;
  size_t second_half;        // where the second copy of [scale, w_i8) starts (calls in HBL_PATH_STREAM_OVERLAP alternate); 0: none
};

ForwardWs carve(int T, int K, int N) {
  ForwardWs w{};
  size_t off = 0;
  w.scale = off;   off = align_up(off + sizeof(float) * (size_t)T, 256);
  w.codesum = off; off = align_up(off + sizeof(int32_t) * (size_t)T, 256);
  const int ts = T < kStreamMaxTokens ? T : kStreamMaxTokens;
  w.zero_region = off;                                      // only the flags must be zero when the contraction starts
  w.counters = off; off += sizeof(int) * align_up(gemm_stream_counter_words(N), 4);
  w.zero_words = (off - w.zero_region) / 4;
  w.acc = off;      off += sizeof(int32_t) * gemm_stream_acc_words(ts, N);
  off = align_up(off, 1024);
  w.codes = off;   off = align_up(off + (size_t)T * K, 1024);
  w.w_i8 = off;    off = align_up(off + (size_t)N * K, 1024);
  if (T <= kStreamMaxTokens) { w.second_half = off; off += w.w_i8; }
  w.total = off;
  return w;
}

// Sets what launch_dependent() reads for the launches of one call, and clears it when the call returns.
struct OverlapScope {
  explicit OverlapScope(bool on) { launch_mode().overlap_ok = on; }
  ~OverlapScope() { launch_mode().overlap_ok = false; launch_mode().releases_early = false; }
};
// SMs a contraction that releases early leaves to the next call's quantizer: its thread blocks come two to an SM.
int overlap_reserve(long act_threads) { return (int)((act_threads + 511) / 512); }

int check_dims(int tokens, int in_dim, int out_dim) {
  if (tokens < 0 || in_dim <= 0 || out_dim <= 0) return HBL_ERR_SHAPE;
  if (in_dim % 128 != 0 || out_dim % 16 != 0) return HBL_ERR_SHAPE;
  if (in_dim > kMaxInDim) return HBL_ERR_TOO_LARGE;
  return HBL_OK;
}

int check_quant_args(int x_dtype, int in_dim, int bits, int use_hadamard, float eps) {
  if (x_dtype != HBL_F32 && x_dtype != HBL_BF16) return HBL_ERR_FORMAT;
  if (bits != 4 && bits != 8) return HBL_ERR_BITS;
  if (!(eps > 0.0f) || !isfinite(eps)) return HBL_ERR_EPS;
  if (use_hadamard && !is_pow2(in_dim)) return HBL_ERR_NOT_POW2;
  return HBL_OK;
}

// Which contraction kernel.  The streaming kernel reads the packed weights once per 128 tokens; the
// large-batch path pays an expansion and a launch per weight tensor.  Measured cross-overs: one pass
// (<= 128 tokens) always goes to the streaming kernel; a single layer of 16 MiB or more of packed weights
// up to 192 tokens, of 32 MiB or more up to 256 (32 MiB: 63 vs 81 us at 256 tokens, 95 vs 92 at 384,
// 126 vs 105 at 512); the seven tensors of a decoder block up to 512 tokens (64 MiB: 237 vs 246 us there).
int resolve_path(int path, int tokens, size_t packed_bytes, int n_tensors) {
  if (path == HBL_PATH_AUTO) {
    if (tokens <= 128) return HBL_PATH_STREAM;
    const int limit = n_tensors > 1 ? kStreamMaxTokens : (packed_bytes >= ((size_t)32 << 20) ? 256 : 192);
    if (tokens <= limit && packed_bytes >= (size_t)16 << 20) return HBL_PATH_STREAM;
    return HBL_PATH_TENSOR;
  }
  if (path == HBL_PATH_STREAM || path == HBL_PATH_STREAM_OVERLAP) return tokens <= kStreamMaxTokens ? path : -1;
  if (path == HBL_PATH_TENSOR || path == HBL_PATH_TENSOR_PACKED) return path;
  return -2;
}

// A side stream per device on which the large-batch path expands packed weights to int8 while the
// caller's stream quantizes activations or runs the previous contraction (the expansion is bound by
// HBM, the contraction by the tensor cores, the quantizer by instruction issue: they overlap well).
// Created on first use; every use forks from the caller's stream and joins it again before returning,
// so in the caller's stream order a call is complete when its last kernel is.
constexpr int kSideEvents = 16;
struct SidePipe {
  bool ready = false;
  cudaStream_t side = nullptr;
  cudaEvent_t fork = nullptr, unpacked[kSideEvents] = {}, consumed[kSideEvents] = {};
};
SidePipe* side_pipe() {
  static SidePipe pipes[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  SidePipe& sp = pipes[dev];
  if (!sp.ready) {
    if (cudaStreamCreateWithFlags(&sp.side, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&sp.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    for (int i = 0; i < kSideEvents; ++i) {
      if (cudaEventCreateWithFlags(&sp.unpacked[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&sp.consumed[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    }
    sp.ready = true;
  }
  return &sp;
}

// quantized activations -> one projection.  Exactly one of y / acc_out set.
int run_gemm(int path, const int8_t* codes, const float* scale, const int32_t* codesum, int T, int K,
             const void* W_packed, int N, const float* alpha, void* y, int32_t* acc_out, int32_t* acc_ws,
             int* counters, int8_t* w_i8, cudaStream_t s) {
  if (path == HBL_PATH_STREAM)
    return launch_gemm_stream(codes, scale, codesum, T, K, W_packed, N, alpha, static_cast<__nv_bfloat16*>(y),
                              acc_out, acc_ws, counters, s);
  int rc = launch_unpack_weights(W_packed, N, K, w_i8, s);
  if (rc != HBL_OK) return rc;
  return launch_gemm_tensor(codes, false, scale, T, K, w_i8, N, alpha, static_cast<__nv_bfloat16*>(y), acc_out, s);
}

}  // namespace

extern "C" {

const char* hbl_status_string(int status) {
  switch (status) {
    case HBL_OK: return "ok";
    case HBL_ERR_NULL: return "null pointer";
    case HBL_ERR_SHAPE: return "unsupported shape";
    case HBL_ERR_NOT_POW2: return "in_dim must be a power of two for the Hadamard transform";
    case HBL_ERR_BITS: return "unsupported bit width";
    case HBL_ERR_ALIGN: return "misaligned pointer";
    case HBL_ERR_WORKSPACE: return "workspace too small";
    case HBL_ERR_EPS: return "eps must be positive and finite";
    case HBL_ERR_CUDA: return "CUDA call failed";
    case HBL_ERR_TIMEOUT: return "device-side wait timed out";
    case HBL_ERR_FORMAT: return "unknown dtype or path";
    case HBL_ERR_TOO_LARGE: return "size beyond the supported maximum";
    default: return "unknown status";
  }
}

size_t hbl_packed_weight_bytes(int out_dim, int in_dim) {
  if (check_dims(0, in_dim, out_dim) != HBL_OK) return 0;
  return (size_t)((out_dim + 127) / 128) * 128 * in_dim / 4;   // rows padded to whole 128-row tiles
}

size_t hbl_workspace_bytes(int max_tokens, int in_dim, int out_dim) {
  if (check_dims(max_tokens, in_dim, out_dim) != HBL_OK) return 0;
  return carve(max_tokens, in_dim, out_dim).total;
}

size_t hbl_quantize_weights_workspace_bytes(int out_dim, int in_dim) {
  if (check_dims(0, in_dim, out_dim) != HBL_OK) return 0;
  return 2048 * sizeof(double);
}

int hbl_quantize_weights(const void* W_latent, int w_dtype, int out_dim, int in_dim, float eps,
                         void* W_packed, float* alpha, void* workspace, size_t workspace_bytes,
                         void* stream) {
  if (!W_latent || !W_packed || !alpha || !workspace) return HBL_ERR_NULL;
  int rc = check_dims(0, in_dim, out_dim);
  if (rc != HBL_OK) return rc;
  if (w_dtype != HBL_F32 && w_dtype != HBL_BF16) return HBL_ERR_FORMAT;
  if (!(eps > 0.0f) || !isfinite(eps)) return HBL_ERR_EPS;
  if (!aligned(W_latent, 16) || !aligned(W_packed, 16) || !aligned(alpha, 4) || !aligned(workspace, 16))
    return HBL_ERR_ALIGN;
  if (workspace_bytes < hbl_quantize_weights_workspace_bytes(out_dim, in_dim)) return HBL_ERR_WORKSPACE;
  return launch_weight_quant(W_latent, w_dtype, out_dim, in_dim, eps, W_packed, alpha, workspace,
                             static_cast<cudaStream_t>(stream));
}

size_t hbl_quantize_weights_rotated_workspace_bytes(int out_dim, int in_dim) {
  const size_t base = hbl_quantize_weights_workspace_bytes(out_dim, in_dim);
  if (base == 0) return 0;
  return align_up(base, 256) + sizeof(float) * (size_t)out_dim * in_dim;
}

int hbl_quantize_weights_rotated(const void* W_latent, int w_dtype, int out_dim, int in_dim, float eps,
                                 void* W_packed, float* alpha, void* workspace, size_t workspace_bytes,
                                 void* stream) {
  if (!W_latent || !W_packed || !alpha || !workspace) return HBL_ERR_NULL;
  int rc = check_dims(0, in_dim, out_dim);
  if (rc != HBL_OK) return rc;
  if (w_dtype != HBL_F32 && w_dtype != HBL_BF16) return HBL_ERR_FORMAT;
  if (!is_pow2(in_dim)) return HBL_ERR_NOT_POW2;
  if (!(eps > 0.0f) || !isfinite(eps)) return HBL_ERR_EPS;
  if (!aligned(W_latent, 16) || !aligned(W_packed, 16) || !aligned(alpha, 4) || !aligned(workspace, 256))
    return HBL_ERR_ALIGN;
  if (workspace_bytes < hbl_quantize_weights_rotated_workspace_bytes(out_dim, in_dim)) return HBL_ERR_WORKSPACE;
  const size_t base = align_up(hbl_quantize_weights_workspace_bytes(out_dim, in_dim), 256);
  float* rotated = reinterpret_cast<float*>(static_cast<char*>(workspace) + base);
  // rows of W H are the transforms of the rows of W (H is symmetric): the activation kernel's transform-only
  // mode, with the weight rows in the place of tokens, then Eq. 1-2 on the result
  rc = launch_act_quant(W_latent, w_dtype, out_dim, in_dim, 4, 1, 1.0f, nullptr, nullptr, nullptr, rotated, nullptr, 0,
                        static_cast<cudaStream_t>(stream));
  if (rc != HBL_OK) return rc;
  return launch_weight_quant(rotated, HBL_F32, out_dim, in_dim, eps, W_packed, alpha, workspace,
                             static_cast<cudaStream_t>(stream));
}

}  // extern "C"

namespace {

// Requirements of the fused normalisation: bf16 input, the transform on, a width the bf16 kernel has.
int check_norm_args(int x_dtype, int in_dim, const void* gain, int gain_dtype, float norm_eps, int tokens) {
  if (x_dtype != HBL_BF16 || (gain_dtype != HBL_F32 && gain_dtype != HBL_BF16)) return HBL_ERR_FORMAT;
  if (!is_pow2(in_dim)) return HBL_ERR_NOT_POW2;
  if (!act_quant_bf16_supported(in_dim)) return HBL_ERR_SHAPE;
  if (!(norm_eps >= 0.0f) || !isfinite(norm_eps)) return HBL_ERR_EPS;
  if (tokens > 0 && !gain) return HBL_ERR_NULL;
  if (!aligned(gain, 16)) return HBL_ERR_ALIGN;
  return HBL_OK;
}

// hbl_forward, hbl_forward_norm (gain != nullptr: normalise first) and hbl_forward_glu (up != nullptr: x is
// the gate projection, the layer's input is SiLU(x) * up).
int forward_impl(const void* x, int x_dtype, const void* gain, int gain_dtype, float norm_eps, const void* up, int tokens,
                 int in_dim,
                 const void* W_packed, const float* alpha, int out_dim, int bits, int use_hadamard, float eps, void* y,
                 void* workspace, size_t workspace_bytes, int path, void* stream) {
  int rc = check_dims(tokens, in_dim, out_dim);
  if (rc != HBL_OK) return rc;
  rc = check_quant_args(x_dtype, in_dim, bits, use_hadamard, eps);
  if (rc != HBL_OK) return rc;
  const int p = resolve_path(path, tokens, (size_t)out_dim * in_dim / 4, 1);
  if (p == -1) return HBL_ERR_TOO_LARGE;
  if (p < 0) return HBL_ERR_FORMAT;
  // INT4 codes two per byte between the two kernels: only on request (measured slower than one code per byte
  // at every size tried: the widening costs the contraction more than the halved code traffic saves)
  const bool packed = (p == HBL_PATH_TENSOR_PACKED);
  if (packed && (bits != 4 || !((gain || up) ? true : act_quant_can_pack(x_dtype, tokens > 64 ? tokens : 65, in_dim, bits, use_hadamard))))
    return HBL_ERR_SHAPE;
  if (tokens == 0) return HBL_OK;
  if (!x || !W_packed || !alpha || !y || !workspace) return HBL_ERR_NULL;
  if (!aligned(x, 16) || !aligned(W_packed, 16) || !aligned(y, 16) || !aligned(workspace, 1024) ||
      !aligned(alpha, 4))
    return HBL_ERR_ALIGN;
  const ForwardWs w = carve(tokens, in_dim, out_dim);
  if (workspace_bytes < w.total) return HBL_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // back-to-back mode: this call's quantizer may run beside the previous call's contraction, so it writes the half
  // of the scratch that call does not read (no slot left to remember the workspace: an ordinary streaming call)
  // The automatic path takes the same mode by itself when it can see that the caller's statement holds: the
  // library's last launch on this stream either does not release early, or writes none of this call's inputs.
  const size_t x_elem = x_dtype == HBL_BF16 ? 2 : 4;
  ByteRange ins[3];
  int n_ins = 0;
  ins[n_ins++] = byte_range(x, (size_t)tokens * in_dim * x_elem);
  if (up) ins[n_ins++] = byte_range(up, (size_t)tokens * in_dim * 2);
  if (gain) ins[n_ins++] = byte_range(gain, (size_t)in_dim * 4);
  const ByteRange outs_written[2] = {byte_range(y, (size_t)tokens * out_dim * 2), byte_range(workspace, w.total)};
  // (the explicit mode is the caller's statement about the inputs; that the workspace is not in use by the call
  //  before is checked either way)
  const bool want_overlap = (p == HBL_PATH_STREAM_OVERLAP && clear_of_last_call(s, ins, 0, outs_written[1])) ||
                            (path == HBL_PATH_AUTO && p == HBL_PATH_STREAM && clear_of_last_call(s, ins, n_ins, outs_written[1]));
  int slot = -1;
  const int half = want_overlap ? next_overlap_half(workspace, &slot) : -1;
  const bool overlap = half >= 0;
  OverlapScope scope(overlap);
  char* ws = static_cast<char*>(workspace) + (half == 1 ? w.second_half : 0);
  float* scale = reinterpret_cast<float*>(ws + w.scale);
  int32_t* codesum = reinterpret_cast<int32_t*>(ws + w.codesum);
  int8_t* codes = reinterpret_cast<int8_t*>(ws + w.codes);
  const bool stream_path = (p == HBL_PATH_STREAM || p == HBL_PATH_STREAM_OVERLAP);
  SidePipe* sp = nullptr;
  int8_t* w_i8 = reinterpret_cast<int8_t*>(static_cast<char*>(workspace) + w.w_i8);
  if (!stream_path) {
    // the weights are expanded on the side stream while the activations are quantized on the caller's
    sp = side_pipe();
    if (sp == nullptr) return HBL_ERR_CUDA;
    HBL_CUDA_OK(cudaEventRecord(sp->fork, s));
    HBL_CUDA_OK(cudaStreamWaitEvent(sp->side, sp->fork, 0));
    rc = launch_unpack_weights(W_packed, out_dim, in_dim, w_i8, sp->side);
    if (rc != HBL_OK) return rc;
    HBL_CUDA_OK(cudaEventRecord(sp->unpacked[0], sp->side));
  }
  int32_t* zf = stream_path ? reinterpret_cast<int32_t*>(ws + w.zero_region) : nullptr;
  const size_t zw = stream_path ? w.zero_words : 0;
  int32_t* cs = stream_path ? codesum : nullptr;             // only the streaming kernel needs the code sums
  if (overlap && !gain && !up && x_dtype == HBL_BF16) {
    // the quantizer whose thread blocks count themselves in, so that the contraction can start on the codes while
    // the call before this one is still draining
    const ActJob job = {x, codes, scale, codesum, in_dim, use_hadamard};
    unsigned* counters = overlap_counters(slot, half);
    if (counters != nullptr && act_multi_bf16_supported(&job, 1)) {
      StreamReady ready = {counters, {0, 0, 0, 0}, counters + 4};
      rc = launch_act_multi_bf16(&job, 1, tokens, bits, eps, zf, zw, s, counters, ready.target);
      if (rc != HBL_OK) return rc;
      rc = launch_gemm_stream(codes, scale, codesum, tokens, in_dim, W_packed, out_dim, alpha,
                              static_cast<__nv_bfloat16*>(y), nullptr, reinterpret_cast<int32_t*>(ws + w.acc),
                              reinterpret_cast<int*>(ws + w.counters), s,
                              overlap_reserve((long)tokens * (in_dim / 64 < 32 ? 32 : in_dim / 64)), &ready);
      if (rc == HBL_OK) record_stream_outputs(s, outs_written, 2);
      return rc;
    }
  }
  rc = gain ? launch_norm_act_quant_bf16(x, gain, gain_dtype, norm_eps, tokens, in_dim, bits, eps, codes, scale, cs, nullptr, zf, zw, s, packed)
       : up ? launch_glu_act_quant_bf16(x, up, tokens, in_dim, bits, eps, codes, scale, cs, nullptr, zf, zw, s, packed)
            : launch_act_quant(x, x_dtype, tokens, in_dim, bits, use_hadamard, eps, codes, scale, cs, nullptr, zf, zw, s, packed);
  if (rc != HBL_OK) {
    if (sp != nullptr) cudaStreamWaitEvent(s, sp->unpacked[0], 0);   // join before reporting the error
    return rc;
  }
  if (stream_path) {
    rc = launch_gemm_stream(codes, scale, codesum, tokens, in_dim, W_packed, out_dim, alpha,
                            static_cast<__nv_bfloat16*>(y), nullptr, reinterpret_cast<int32_t*>(ws + w.acc),
                            reinterpret_cast<int*>(ws + w.counters), s,
                            overlap ? overlap_reserve((long)tokens * (in_dim / 64 < 32 ? 32 : in_dim / 64)) : -1);
    if (overlap && rc == HBL_OK) record_stream_outputs(s, outs_written, 2);
    return rc;
  }
  HBL_CUDA_OK(cudaStreamWaitEvent(s, sp->unpacked[0], 0));
  return launch_gemm_tensor(codes, packed, scale, tokens, in_dim, w_i8, out_dim, alpha, static_cast<__nv_bfloat16*>(y), nullptr, s);
}

}  // namespace

extern "C" {

int hbl_forward(const void* x, int x_dtype, int tokens, int in_dim, const void* W_packed,
                const float* alpha, int out_dim, int bits, int use_hadamard, float eps, void* y,
                void* workspace, size_t workspace_bytes, int path, void* stream) {
  return forward_impl(x, x_dtype, nullptr, HBL_F32, 0.f, nullptr, tokens, in_dim, W_packed, alpha, out_dim, bits, use_hadamard, eps,
                      y, workspace, workspace_bytes, path, stream);
}

int hbl_forward_norm(const void* x, const void* gain, int gain_dtype, float norm_eps, int tokens, int in_dim,
                     const void* W_packed, const float* alpha, int out_dim, int bits, float eps, void* y, void* workspace,
                     size_t workspace_bytes, int path, void* stream) {
  const int rc = check_norm_args(HBL_BF16, in_dim, gain, gain_dtype, norm_eps, tokens);
  if (rc != HBL_OK) return rc;
  return forward_impl(x, HBL_BF16, gain, gain_dtype, norm_eps, nullptr, tokens, in_dim, W_packed, alpha, out_dim, bits, 1, eps, y,
                      workspace, workspace_bytes, path, stream);
}

int hbl_forward_glu(const void* gate, const void* up, int tokens, int in_dim, const void* W_packed, const float* alpha,
                    int out_dim, int bits, float eps, void* y, void* workspace, size_t workspace_bytes, int path,
                    void* stream) {
  if (!is_pow2(in_dim)) return HBL_ERR_NOT_POW2;
  if (!act_quant_bf16_supported(in_dim)) return HBL_ERR_SHAPE;
  if (tokens > 0 && !up) return HBL_ERR_NULL;
  if (!aligned(up, 16)) return HBL_ERR_ALIGN;
  return forward_impl(gate, HBL_BF16, nullptr, HBL_F32, 0.f, up, tokens, in_dim, W_packed, alpha, out_dim, bits, 1, eps, y,
                      workspace, workspace_bytes, path, stream);
}

int hbl_glu_quantize_act(const void* gate, const void* up, int tokens, int in_dim, int bits, float eps,
                         int8_t* codes_out, float* scale_out, int32_t* codesum_out, float* xr_out, void* stream) {
  int rc = check_dims(tokens, in_dim, 16);
  if (rc != HBL_OK) return rc;
  rc = check_quant_args(HBL_BF16, in_dim, bits, 1, eps);
  if (rc != HBL_OK) return rc;
  if (!act_quant_bf16_supported(in_dim)) return HBL_ERR_SHAPE;
  if (tokens == 0) return HBL_OK;
  if (!gate || !up) return HBL_ERR_NULL;
  if (!aligned(gate, 16) || !aligned(up, 16)) return HBL_ERR_ALIGN;
  if (xr_out == nullptr) {
    if (!codes_out || !scale_out) return HBL_ERR_NULL;
    if (!aligned(codes_out, 16)) return HBL_ERR_ALIGN;
  } else if (!aligned(xr_out, 16)) {
    return HBL_ERR_ALIGN;
  }
  return launch_glu_act_quant_bf16(gate, up, tokens, in_dim, bits, eps, codes_out, scale_out, codesum_out, xr_out,
                                   nullptr, 0, static_cast<cudaStream_t>(stream));
}

int hbl_norm_quantize_act(const void* x, const void* gain, int gain_dtype, float norm_eps, int tokens, int in_dim,
                          int bits, float eps, int8_t* codes_out, float* scale_out, int32_t* codesum_out, float* xr_out,
                          void* stream) {
  int rc = check_dims(tokens, in_dim, 16);
  if (rc != HBL_OK) return rc;
  rc = check_quant_args(HBL_BF16, in_dim, bits, 1, eps);
  if (rc != HBL_OK) return rc;
  rc = check_norm_args(HBL_BF16, in_dim, gain, gain_dtype, norm_eps, tokens);
  if (rc != HBL_OK) return rc;
  if (tokens == 0) return HBL_OK;
  if (!x) return HBL_ERR_NULL;
  if (!aligned(x, 16)) return HBL_ERR_ALIGN;
  if (xr_out == nullptr) {
    if (!codes_out || !scale_out) return HBL_ERR_NULL;
    if (!aligned(codes_out, 16)) return HBL_ERR_ALIGN;
  } else if (!aligned(xr_out, 16)) {
    return HBL_ERR_ALIGN;
  }
  return launch_norm_act_quant_bf16(x, gain, gain_dtype, norm_eps, tokens, in_dim, bits, eps, codes_out, scale_out, codesum_out,
                                    xr_out, nullptr, 0, static_cast<cudaStream_t>(stream));
}

// ---- decoder block: four quantizations, seven projections -------------------------------
namespace {
struct BlockWs {
  size_t scale[4], codesum[4], codes[4], zero_region, counters[7], acc[7], w_i8, total, zero_words;
  size_t second_half;        // as in ForwardWs
};
BlockWs carve_block(int T, int H, int F) {
  BlockWs w{};
  const int in_dims[4] = {H, H, H, F};                       // attn_in, o_in, ffn_in, down_in
  const int out_dims[7] = {H, H, H, H, F, F, H};             // q k v o up gate down
  size_t off = 0;
  for (int i = 0; i < 4; ++i) { w.scale[i] = off; off = align_up(off + 4 * (size_t)T, 256); }
  for (int i = 0; i < 4; ++i) { w.codesum[i] = off; off = align_up(off + 4 * (size_t)T, 256); }
  const int ts = T < kStreamMaxTokens ? T : kStreamMaxTokens;
  w.zero_region = off;                                      // the seven flag arrays first: only they must be zero
  for (int i = 0; i < 7; ++i) { w.counters[i] = off; off += sizeof(int) * align_up(gemm_stream_counter_words(out_dims[i]), 4); }
  w.zero_words = (off - w.zero_region) / 4;
  for (int i = 0; i < 7; ++i) { w.acc[i] = off; off += sizeof(int32_t) * gemm_stream_acc_words(ts, out_dims[i]); }
  off = align_up(off, 1024);
  for (int i = 0; i < 4; ++i) { w.codes[i] = off; off = align_up(off + (size_t)T * in_dims[i], 1024); }
  w.w_i8 = off; off = align_up(off + 3 * align_up((size_t)F * H, 1024), 1024);   // three buffers of the largest weight (F x H)
  if (T <= kStreamMaxTokens) { w.second_half = off; off += w.w_i8; }
  w.total = off;
  return w;
}
}  // namespace

size_t hbl_block_workspace_bytes(int max_tokens, int hidden, int ffn) {
  if (check_dims(max_tokens, hidden, hidden) != HBL_OK || check_dims(max_tokens, ffn, ffn) != HBL_OK) return 0;
  return carve_block(max_tokens, hidden, ffn).total;
}

int hbl_block_forward(const hbl_block_t* b, void* workspace, size_t workspace_bytes, int path, void* stream) {
  if (!b) return HBL_ERR_NULL;
  const int T = b->tokens, H = b->hidden, F = b->ffn;
  int rc = check_dims(T, H, H);
  if (rc != HBL_OK) return rc;
  rc = check_dims(T, F, F);
  if (rc != HBL_OK) return rc;
  rc = check_quant_args(b->x_dtype, H, b->bits, 1, b->eps);
  if (rc != HBL_OK) return rc;
  if (!is_pow2(F)) return HBL_ERR_NOT_POW2;
  const int p = resolve_path(path, T, ((size_t)4 * H * H + (size_t)3 * H * F) / 4, 7);
  if (p == -1) return HBL_ERR_TOO_LARGE;
  if (p < 0) return HBL_ERR_FORMAT;
  if (p == HBL_PATH_TENSOR_PACKED && b->bits != 4) return HBL_ERR_SHAPE;
  if (T == 0) return HBL_OK;
  const void* xs[4] = {b->x_attn_in, b->x_o_in, b->x_ffn_in, b->x_down_in};
  const void* Ws[7] = {b->Wq, b->Wk, b->Wv, b->Wo, b->Wup, b->Wgate, b->Wdown};
  void* ys[7] = {b->yq, b->yk, b->yv, b->yo, b->yup, b->ygate, b->ydown};
  // x_down_in == NULL: the feed-forward block is chained for real -- the down projection's input is
  // SiLU(ygate) * yup, formed inside its activation kernel from the two outputs written by this call
  const bool chain_ffn = (b->x_down_in == nullptr);
  if (chain_ffn && !act_quant_bf16_supported(F)) return HBL_ERR_SHAPE;
  for (int i = 0; i < (chain_ffn ? 3 : 4); ++i) {
    if (!xs[i]) return HBL_ERR_NULL;
    if (!aligned(xs[i], 16)) return HBL_ERR_ALIGN;
  }
  for (int i = 0; i < 7; ++i) {
    if (!Ws[i] || !ys[i]) return HBL_ERR_NULL;
    if (!aligned(Ws[i], 16) || !aligned(ys[i], 16)) return HBL_ERR_ALIGN;
  }
  if (!b->alpha7 || !workspace) return HBL_ERR_NULL;
  if (!aligned(workspace, 1024)) return HBL_ERR_ALIGN;
  const BlockWs w = carve_block(T, H, F);
  if (workspace_bytes < w.total) return HBL_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // back-to-back mode (not for the chained feed-forward block, whose second quantizer reads the first launch's
  // outputs): see forward_impl
  const size_t x_elem = b->x_dtype == HBL_BF16 ? 2 : 4;
  ByteRange ins[4];
  for (int i = 0; i < 4; ++i) ins[i] = byte_range(xs[i], xs[i] ? (size_t)T * (i == 3 ? F : H) * x_elem : 0);
  const ByteRange ws_range = byte_range(workspace, w.total);
  const bool want_overlap = !chain_ffn && ((p == HBL_PATH_STREAM_OVERLAP && clear_of_last_call(s, ins, 0, ws_range)) ||
                                           (path == HBL_PATH_AUTO && p == HBL_PATH_STREAM && clear_of_last_call(s, ins, 4, ws_range)));
  int slot = -1;
  const int half = want_overlap ? next_overlap_half(workspace, &slot) : -1;
  const bool overlap = half >= 0;
  OverlapScope scope(overlap);
  char* ws = static_cast<char*>(workspace) + (half == 1 ? w.second_half : 0);
  const int in_dims[4] = {H, H, H, F};
  const int had[4] = {0, 1, 0, 1};
  const bool stream_path = (p == HBL_PATH_STREAM || p == HBL_PATH_STREAM_OVERLAP);
  SidePipe* sp = nullptr;
  if (!stream_path) {
    // fork the side stream now: its first expansions overlap the quantizations below, and it starts
    // after whatever the caller queued before (an earlier call may still be reading the int8 buffers)
    sp = side_pipe();
    if (sp == nullptr) return HBL_ERR_CUDA;
    HBL_CUDA_OK(cudaEventRecord(sp->fork, s));
    HBL_CUDA_OK(cudaStreamWaitEvent(sp->side, sp->fork, 0));
  }
  bool packed[4] = {false, false, false, false};              // on request: INT4 codes two per byte where the kernel can
  for (int i = 0; i < 4; ++i)
    packed[i] = p == HBL_PATH_TENSOR_PACKED && b->bits == 4 &&
                ((i == 3 && chain_ffn) ? true : act_quant_can_pack(b->x_dtype, T, in_dims[i], b->bits, had[i]));
  // small batch, bf16 inputs: one launch quantizes all inputs (each launch is a dependent step of a microsecond
  // or two, which is what a call of a few tokens spends most of its time on besides the weights)
  const int n_act = chain_ffn ? 3 : 4;
  bool one_launch = false;
  StreamReady ready = {nullptr, {0, 0, 0, 0}, nullptr};     // back-to-back mode: the quantizer's thread blocks count themselves in
  if (stream_path && b->x_dtype == HBL_BF16) {
    ActJob aj[4];
    for (int i = 0; i < n_act; ++i)
      aj[i] = {xs[i], reinterpret_cast<int8_t*>(ws + w.codes[i]), reinterpret_cast<float*>(ws + w.scale[i]),
               reinterpret_cast<int32_t*>(ws + w.codesum[i]), in_dims[i], had[i]};
    if (act_multi_bf16_supported(aj, n_act)) {
      unsigned* counters = overlap ? overlap_counters(slot, half) : nullptr;
      if (counters != nullptr) ready = {counters, {0, 0, 0, 0}, counters + 4};
      rc = launch_act_multi_bf16(aj, n_act, T, b->bits, b->eps, reinterpret_cast<int32_t*>(ws + w.zero_region),
                                 w.zero_words, s, counters, ready.target);
      if (rc != HBL_OK) return rc;
      one_launch = true;
    }
  }
  for (int i = 0; i < (one_launch ? 0 : n_act); ++i) {
    rc = launch_act_quant(xs[i], b->x_dtype, T, in_dims[i], b->bits, had[i], b->eps,
                          reinterpret_cast<int8_t*>(ws + w.codes[i]), reinterpret_cast<float*>(ws + w.scale[i]),
                          stream_path ? reinterpret_cast<int32_t*>(ws + w.codesum[i]) : nullptr, nullptr,
                          (stream_path && i == 0) ? reinterpret_cast<int32_t*>(ws + w.zero_region) : nullptr,
                          (stream_path && i == 0) ? w.zero_words : 0, s, packed[i]);
    if (rc != HBL_OK) return rc;
  }
  const int src[7] = {0, 0, 0, 1, 2, 2, 3};                  // which quantized input feeds each projection
  const int out_dims[7] = {H, H, H, H, F, F, H};
  if (stream_path) {
    // small batch: all seven weight tensors stream through one launch
    StreamInput inputs[4];
    for (int i = 0; i < 4; ++i)
      inputs[i] = {reinterpret_cast<int8_t*>(ws + w.codes[i]), reinterpret_cast<float*>(ws + w.scale[i]),
                   reinterpret_cast<int32_t*>(ws + w.codesum[i]), in_dims[i]};
    StreamJob jobs[7];
    for (int i = 0; i < 7; ++i)
      jobs[i] = {Ws[i], b->alpha7 + i, static_cast<__nv_bfloat16*>(ys[i]), nullptr, out_dims[i], src[i]};
    int32_t* part = reinterpret_cast<int32_t*>(ws + w.acc[0]);
    int* flags = reinterpret_cast<int*>(ws + w.counters[0]);
    if (!chain_ffn) {
      long act_threads = 0;                                   // of the next call's quantizer, which has this call's shape
      for (int i = 0; i < 4; ++i) act_threads += (long)T * (in_dims[i] / 64);
      rc = launch_gemm_stream_multi(inputs, 4, jobs, 7, T, part, flags, s, overlap ? overlap_reserve(act_threads) : -1,
                                    ready.ready != nullptr ? &ready : nullptr);
      if (overlap && rc == HBL_OK) {
        ByteRange written[8];
        for (int i = 0; i < 7; ++i) written[i] = byte_range(ys[i], (size_t)T * out_dims[i] * 2);
        written[7] = byte_range(workspace, w.total);
        record_stream_outputs(s, written, 8);
      }
      return rc;
    }
    // chained: six projections, then the gating product + quantizer (which also clears the flags again: it
    // starts only when the first launch has completed), then the down projection
    rc = launch_gemm_stream_multi(inputs, 3, jobs, 6, T, part, flags, s);
    if (rc != HBL_OK) return rc;
    rc = launch_glu_act_quant_bf16(ys[5], ys[4], T, F, b->bits, b->eps, reinterpret_cast<int8_t*>(ws + w.codes[3]),
                                   reinterpret_cast<float*>(ws + w.scale[3]), reinterpret_cast<int32_t*>(ws + w.codesum[3]),
                                   nullptr, reinterpret_cast<int32_t*>(ws + w.zero_region), w.zero_words, s);
    if (rc != HBL_OK) return rc;
    StreamJob down = jobs[6];
    down.input = 0;
    return launch_gemm_stream_multi(&inputs[3], 1, &down, 1, T, part, flags, s);
  }
  const size_t buf_bytes = align_up((size_t)F * H, 1024);
  if (T <= kFuseMaxTokens && H % 256 == 0 && F % 256 == 0 && 4 * (size_t)H <= (size_t)F) {
    // Large batch, fused: q | k | v share one quantized input and so do up | gate, so each group is ONE contraction
    // over the concatenated weight rows (per-output alpha and output tensor in the epilogue): four launches
    // instead of seven, and fewer partly filled waves of tiles.  Measured on the 7B shapes, same box, fused vs
    // seven launches: 0.310 vs 0.313 ms at 1024 tokens, 0.963 vs 0.960 at 4096, 3.82 vs 3.70 at 16384 (a
    // contraction over 32768 concatenated rows keeps fewer weight tiles in L2 per token block than two over
    // 16384): so only up to kFuseMaxTokens tokens.  Int8 weights: up | gate fill buffers 0 and 1,
    // q | k | v | o share buffer 2, which `down` reuses once their contractions are done; all expansions run on
    // the side stream underneath the quantizers and the contractions before them.
    int8_t* buf01 = reinterpret_cast<int8_t*>(ws + w.w_i8);
    int8_t* buf2 = buf01 + 2 * buf_bytes;
    int8_t* w_dst[7] = {buf2, buf2 + (size_t)H * H, buf2 + 2 * (size_t)H * H, buf2 + 3 * (size_t)H * H,
                        buf01, buf01 + (size_t)F * H, buf2};
    const int first[4] = {0, 3, 4, 6}, count[4] = {3, 1, 2, 1};
    auto expand_group = [&](int g) -> int {                   // the group's tensors to int8, on the side stream
      for (int i = first[g]; i < first[g] + count[g]; ++i) {
        const int r = launch_unpack_weights(Ws[i], out_dims[i], in_dims[src[i]], w_dst[i], sp->side);
        if (r != HBL_OK) return r;
      }
      return cudaEventRecord(sp->unpacked[g], sp->side) == cudaSuccess ? HBL_OK : HBL_ERR_CUDA;
    };
    for (int g = 0; g < 3; ++g) {
      rc = expand_group(g);
      if (rc != HBL_OK) return rc;
    }
    for (int g = 0; g < 4; ++g) {
      const int i0 = first[g], xi = src[i0];
      if (g == 2) {
        // `down` overwrites q | k | v | o: its expansion is queued now that their contractions are (events recorded
        // above), and runs underneath the up | gate contraction
        HBL_CUDA_OK(cudaStreamWaitEvent(sp->side, sp->consumed[0], 0));
        HBL_CUDA_OK(cudaStreamWaitEvent(sp->side, sp->consumed[1], 0));
        rc = expand_group(3);
        if (rc != HBL_OK) return rc;
      }
      HBL_CUDA_OK(cudaStreamWaitEvent(s, sp->unpacked[g], 0));
      if (chain_ffn && g == 3) {                              // up and gate are complete in stream order
        rc = launch_glu_act_quant_bf16(ys[5], ys[4], T, F, b->bits, b->eps, reinterpret_cast<int8_t*>(ws + w.codes[3]),
                                       reinterpret_cast<float*>(ws + w.scale[3]), nullptr, nullptr, nullptr, 0, s, packed[3]);
        if (rc != HBL_OK) return rc;
      }
      TensorOutputs outs = {};
      outs.n = count[g];
      int begin = 0;
      for (int j = 0; j < count[g]; ++j) {
        outs.begin[j] = begin; outs.width[j] = out_dims[i0 + j];
        outs.y[j] = static_cast<__nv_bfloat16*>(ys[i0 + j]); outs.alpha[j] = b->alpha7 + i0 + j;
        begin += out_dims[i0 + j];
      }
      rc = launch_gemm_tensor_multi(reinterpret_cast<int8_t*>(ws + w.codes[xi]), packed[xi], reinterpret_cast<float*>(ws + w.scale[xi]),
                                    T, in_dims[xi], w_dst[i0], outs, nullptr, s);
      if (rc != HBL_OK) return rc;
      if (g < 2) HBL_CUDA_OK(cudaEventRecord(sp->consumed[g], s));
    }
    return HBL_OK;
  }
  // Large batch, other shapes: tensor i+1 is expanded to int8 on the side stream (two buffers alternate) while
  // tensor i is contracted on the caller's stream.
  for (int i = 0; i < 7 && rc == HBL_OK; ++i) {
    const int xi = src[i];
    int8_t* w_i8 = reinterpret_cast<int8_t*>(ws + w.w_i8 + (size_t)(i & 1) * buf_bytes);
    if (i >= 2) HBL_CUDA_OK(cudaStreamWaitEvent(sp->side, sp->consumed[i - 2], 0));   // the buffer's previous reader
    rc = launch_unpack_weights(Ws[i], out_dims[i], in_dims[xi], w_i8, sp->side);
    if (rc != HBL_OK) break;
    HBL_CUDA_OK(cudaEventRecord(sp->unpacked[i], sp->side));
    HBL_CUDA_OK(cudaStreamWaitEvent(s, sp->unpacked[i], 0));
    if (chain_ffn && i == 6) {                                // up and gate are complete in stream order
      rc = launch_glu_act_quant_bf16(ys[5], ys[4], T, F, b->bits, b->eps, reinterpret_cast<int8_t*>(ws + w.codes[3]),
                                     reinterpret_cast<float*>(ws + w.scale[3]), nullptr, nullptr, nullptr, 0, s, packed[3]);
      if (rc != HBL_OK) break;
    }
    rc = launch_gemm_tensor(reinterpret_cast<int8_t*>(ws + w.codes[xi]), packed[xi], reinterpret_cast<float*>(ws + w.scale[xi]), T,
                            in_dims[xi], w_i8, out_dims[i], b->alpha7 + i, static_cast<__nv_bfloat16*>(ys[i]), nullptr, s);
    if (rc != HBL_OK) break;
    HBL_CUDA_OK(cudaEventRecord(sp->consumed[i], s));
  }
  return rc;
}

unsigned long long hbl_launch_count(void) { return g_launches; }

int hbl_profile_events(void** start_events, void** stop_events, int n, int kernel) {
  if (n < 0 || kernel < 0 || kernel > KERNEL_WEIGHT) return -HBL_ERR_SHAPE;
  if (n > 0 && kernel != 0 && (!start_events || !stop_events)) return -HBL_ERR_NULL;
  if (kernel == 0) {                                          // everything off
    int used = 0;
    for (Profile& pr : g_prof) { used += pr.next; pr = Profile(); }
    return used;
  }
  Profile& pr = g_prof[kernel];
  const int used = pr.next;
  pr = Profile();
  if (n > 0) { pr.starts = start_events; pr.stops = stop_events; pr.n = n; }
  return used;
}

namespace {

// Side streams and events of hbl_forward_host, created on first use, one set per device.
constexpr int kHostMaxChunks = 16;
constexpr int kHostChunkTokens = 2048;
struct HostPipe {
  bool ready = false;
  cudaStream_t copy_in = nullptr, copy_out = nullptr;
  cudaEvent_t start = nullptr, out_done = nullptr, in_done[kHostMaxChunks] = {}, comp_done[kHostMaxChunks] = {};
};
HostPipe* host_pipe() {
  static HostPipe pipes[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  HostPipe& hp = pipes[dev];
  if (!hp.ready) {
    if (cudaStreamCreateWithFlags(&hp.copy_in, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithFlags(&hp.copy_out, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&hp.out_done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    for (int c = 0; c < kHostMaxChunks; ++c) {
      if (cudaEventCreateWithFlags(&hp.in_done[c], cudaEventDisableTiming) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&hp.comp_done[c], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    }
    hp.ready = true;
  }
  return &hp;
}

}  // namespace

int hbl_forward_host(const void* x_host, int x_dtype, int tokens, int in_dim, const void* W_packed,
                     const float* alpha, int out_dim, int bits, int use_hadamard, float eps, void* y_host,
                     void* x_stage, void* y_stage, void* workspace, size_t workspace_bytes, int path,
                     void* stream) {
  if (tokens < 0) return HBL_ERR_SHAPE;
  if (tokens > 0 && (!x_host || !y_host || !x_stage || !y_stage)) return HBL_ERR_NULL;
  if (x_dtype != HBL_F32 && x_dtype != HBL_BF16) return HBL_ERR_FORMAT;
  int rc = check_dims(tokens, in_dim, out_dim);
  if (rc != HBL_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t x_row = (size_t)in_dim * (x_dtype == HBL_F32 ? 4 : 2), y_row = (size_t)out_dim * 2;
  if (tokens <= kHostChunkTokens) {
    // small calls: copy in, run, copy out, all in order on the caller's stream
    if (tokens > 0) HBL_CUDA_OK(cudaMemcpyAsync(x_stage, x_host, x_row * tokens, cudaMemcpyHostToDevice, s));
    rc = hbl_forward(x_stage, x_dtype, tokens, in_dim, W_packed, alpha, out_dim, bits, use_hadamard, eps,
                     y_stage, workspace, workspace_bytes, path, stream);
    if (rc != HBL_OK) return rc;
    if (tokens > 0) HBL_CUDA_OK(cudaMemcpyAsync(y_host, y_stage, y_row * tokens, cudaMemcpyDeviceToHost, s));
    return HBL_OK;
  }
  // Large calls run as a pipeline over chunks of tokens (rows are independent, Eq. 3-7 are per token):
  // chunk c+1 crosses the bus on one side stream while chunk c is computed on the caller's stream and
  // chunk c-1 returns on the other side stream, so the call costs about what its larger copy costs.
  HostPipe* hp = host_pipe();
  if (hp == nullptr) return HBL_ERR_CUDA;
  int chunk = kHostChunkTokens;
  if ((tokens + chunk - 1) / chunk > kHostMaxChunks) chunk = ((tokens + kHostMaxChunks - 1) / kHostMaxChunks + 127) / 128 * 128;
  const int n_chunks = (tokens + chunk - 1) / chunk;
  HBL_CUDA_OK(cudaEventRecord(hp->start, s));                 // what the caller queued before (it may still use the stages)
  HBL_CUDA_OK(cudaStreamWaitEvent(hp->copy_in, hp->start, 0));
  HBL_CUDA_OK(cudaStreamWaitEvent(hp->copy_out, hp->start, 0));
  for (int c = 0; c < n_chunks; ++c) {
    const int t0 = c * chunk, tn = tokens - t0 < chunk ? tokens - t0 : chunk;
    const char* xh = static_cast<const char*>(x_host) + x_row * t0;
    char* xd = static_cast<char*>(x_stage) + x_row * t0;
    char* yd = static_cast<char*>(y_stage) + y_row * t0;
    char* yh = static_cast<char*>(y_host) + y_row * t0;
    HBL_CUDA_OK(cudaMemcpyAsync(xd, xh, x_row * tn, cudaMemcpyHostToDevice, hp->copy_in));
    HBL_CUDA_OK(cudaEventRecord(hp->in_done[c], hp->copy_in));
    HBL_CUDA_OK(cudaStreamWaitEvent(s, hp->in_done[c], 0));
    rc = hbl_forward(xd, x_dtype, tn, in_dim, W_packed, alpha, out_dim, bits, use_hadamard, eps, yd, workspace,
                     workspace_bytes, path, stream);
    if (rc != HBL_OK) return rc;
    HBL_CUDA_OK(cudaEventRecord(hp->comp_done[c], s));
    HBL_CUDA_OK(cudaStreamWaitEvent(hp->copy_out, hp->comp_done[c], 0));
    HBL_CUDA_OK(cudaMemcpyAsync(yh, yd, y_row * tn, cudaMemcpyDeviceToHost, hp->copy_out));
  }
  HBL_CUDA_OK(cudaEventRecord(hp->out_done, hp->copy_out));
  HBL_CUDA_OK(cudaStreamWaitEvent(s, hp->out_done, 0));       // the call is complete, in the caller's stream order, when y_host is
  return HBL_OK;
}

int hbl_check_status(void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(s) != cudaSuccess) return HBL_ERR_CUDA;
  int* word = device_status_word();
  if (word == nullptr) return HBL_ERR_CUDA;
  int st = 0;
  if (cudaMemcpy(&st, word, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return HBL_ERR_CUDA;
  if (st != 0 && cudaMemset(word, 0, sizeof(int)) != cudaSuccess) return HBL_ERR_CUDA;
  if (st != 0) {
    // a kernel that gave up may have left the back-to-back mode's counters mid-count: back to zero (the stream was
    // synchronised above; calls on other streams of this device must not be in flight, as for the status word)
    unsigned* counters = overlap_counters(0, 0);
    if (counters == nullptr || cudaMemset(counters, 0, sizeof(unsigned) * kWorkspaceSlots * 2 * 8) != cudaSuccess) return HBL_ERR_CUDA;
  }
  return st;
}

int hbl_hadamard_f32(const void* x, int x_dtype, int tokens, int in_dim, float* xr_out, void* stream) {
  int rc = check_dims(tokens, in_dim, 16);
  if (rc != HBL_OK) return rc;
  if (x_dtype != HBL_F32 && x_dtype != HBL_BF16) return HBL_ERR_FORMAT;
  if (!is_pow2(in_dim)) return HBL_ERR_NOT_POW2;
  if (tokens == 0) return HBL_OK;
  if (!x || !xr_out) return HBL_ERR_NULL;
  if (!aligned(x, 16) || !aligned(xr_out, 16)) return HBL_ERR_ALIGN;
  return launch_act_quant(x, x_dtype, tokens, in_dim, 4, 1, 1.0f, nullptr, nullptr, nullptr, xr_out, nullptr, 0,
                          static_cast<cudaStream_t>(stream));
}

int hbl_hadamard_bf16(const void* g, int tokens, int in_dim, void* out, void* stream) {
  int rc = check_dims(tokens, in_dim, 16);
  if (rc != HBL_OK) return rc;
  if (!is_pow2(in_dim)) return HBL_ERR_NOT_POW2;
  if (in_dim < 2048 || in_dim > 16384) return HBL_ERR_SHAPE;
  if (tokens == 0) return HBL_OK;
  if (!g || !out) return HBL_ERR_NULL;
  if (!aligned(g, 16) || !aligned(out, 16)) return HBL_ERR_ALIGN;
  return launch_hadamard_bf16(g, tokens, in_dim, out, static_cast<cudaStream_t>(stream));
}

int hbl_quantize_act(const void* x, int x_dtype, int tokens, int in_dim, int bits, int use_hadamard,
                     float eps, int8_t* codes_out, float* scale_out, int32_t* codesum_out, void* stream) {
  int rc = check_dims(tokens, in_dim, 16);
  if (rc != HBL_OK) return rc;
  rc = check_quant_args(x_dtype, in_dim, bits, use_hadamard, eps);
  if (rc != HBL_OK) return rc;
  if (tokens == 0) return HBL_OK;
  if (!x || !codes_out || !scale_out) return HBL_ERR_NULL;
  if (!aligned(x, 16) || !aligned(codes_out, 16) || !aligned(scale_out, 4)) return HBL_ERR_ALIGN;
  return launch_act_quant(x, x_dtype, tokens, in_dim, bits, use_hadamard, eps, codes_out, scale_out, codesum_out,
                          nullptr, nullptr, 0, static_cast<cudaStream_t>(stream));
}

int hbl_quantize_act_int4_packed(const void* x, int x_dtype, int tokens, int in_dim, int use_hadamard, float eps,
                                 uint8_t* codes_packed, float* scale_out, void* stream) {
  int rc = check_dims(tokens, in_dim, 16);
  if (rc != HBL_OK) return rc;
  rc = check_quant_args(x_dtype, in_dim, 4, use_hadamard, eps);
  if (rc != HBL_OK) return rc;
  if (!act_quant_can_pack(x_dtype, tokens > 64 ? tokens : 65, in_dim, 4, use_hadamard)) return HBL_ERR_SHAPE;
  if (tokens == 0) return HBL_OK;
  if (tokens <= 64 && !use_hadamard) return HBL_ERR_SHAPE;    // the small-batch kernels write one code per byte
  if (!x || !codes_packed || !scale_out) return HBL_ERR_NULL;
  if (!aligned(x, 16) || !aligned(codes_packed, 16) || !aligned(scale_out, 4)) return HBL_ERR_ALIGN;
  return launch_act_quant(x, x_dtype, tokens, in_dim, 4, use_hadamard, eps, reinterpret_cast<int8_t*>(codes_packed), scale_out,
                          nullptr, nullptr, nullptr, 0, static_cast<cudaStream_t>(stream), true);
}

int hbl_gemm_i32_int4_packed(const uint8_t* codes_packed, int tokens, int in_dim, const void* W_packed, int out_dim,
                             int32_t* acc_out, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = check_dims(tokens, in_dim, out_dim);
  if (rc != HBL_OK) return rc;
  if (tokens == 0) return HBL_OK;
  if (!codes_packed || !W_packed || !acc_out || !workspace) return HBL_ERR_NULL;
  if (!aligned(codes_packed, 16) || !aligned(W_packed, 16) || !aligned(acc_out, 16) || !aligned(workspace, 1024))
    return HBL_ERR_ALIGN;
  const ForwardWs w = carve(tokens, in_dim, out_dim);
  if (workspace_bytes < w.total) return HBL_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int8_t* w_i8 = reinterpret_cast<int8_t*>(static_cast<char*>(workspace) + w.w_i8);
  rc = launch_unpack_weights(W_packed, out_dim, in_dim, w_i8, s);
  if (rc != HBL_OK) return rc;
  return launch_gemm_tensor(codes_packed, true, nullptr, tokens, in_dim, w_i8, out_dim, nullptr, nullptr, acc_out, s);
}

int hbl_gemm_i32(const int8_t* codes, const int32_t* codesum, int tokens, int in_dim, const void* W_packed,
                 int out_dim, int32_t* acc_out, void* workspace, size_t workspace_bytes, int path, void* stream) {
  int rc = check_dims(tokens, in_dim, out_dim);
  if (rc != HBL_OK) return rc;
  const int p = resolve_path(path, tokens, (size_t)out_dim * in_dim / 4, 1);
  if (p == -1) return HBL_ERR_TOO_LARGE;
  if (p < 0 || p == HBL_PATH_STREAM_OVERLAP) return HBL_ERR_FORMAT;   // (the caller's codes: nothing here to run beside a previous call)
  if (tokens == 0) return HBL_OK;
  if (!codes || !W_packed || !acc_out || !workspace) return HBL_ERR_NULL;
  if (p == HBL_PATH_TENSOR_PACKED) return HBL_ERR_FORMAT;      // these codes are one per byte: see hbl_gemm_i32_int4_packed
  if (p == HBL_PATH_STREAM && !codesum) return HBL_ERR_NULL;
  if (!aligned(codes, 16) || !aligned(W_packed, 16) || !aligned(acc_out, 16) || !aligned(workspace, 1024))
    return HBL_ERR_ALIGN;
  const ForwardWs w = carve(tokens, in_dim, out_dim);
  if (workspace_bytes < w.total) return HBL_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  if (p == HBL_PATH_STREAM) HBL_CUDA_OK(cudaMemsetAsync(ws + w.zero_region, 0, w.zero_words * 4, s));
  return run_gemm(p, codes, nullptr, codesum, tokens, in_dim, W_packed, out_dim, nullptr, nullptr, acc_out,
                  reinterpret_cast<int32_t*>(ws + w.acc), reinterpret_cast<int*>(ws + w.counters),
                  reinterpret_cast<int8_t*>(ws + w.w_i8), s);
}

size_t hbl_kv_codes_bytes(int tokens, int n_heads, int head_dim, int bits) {
  if (tokens < 0 || n_heads <= 0 || (head_dim != 64 && head_dim != 128 && head_dim != 256)) return 0;
  if (bits != 3 && bits != 4 && bits != 8) return 0;
  return (size_t)tokens * n_heads * head_dim * bits / 8;
}

int hbl_quantize_kv(const void* x, int tokens, int n_heads, int head_dim, int bits, int seq_len, float eps, void* codes,
                    float* scale, void* bos_codes, float* bos_scale, void* stream) {
  if (tokens < 0 || n_heads <= 0) return HBL_ERR_SHAPE;
  if (head_dim != 64 && head_dim != 128 && head_dim != 256) return HBL_ERR_SHAPE;
  if (bits != 3 && bits != 4 && bits != 8) return HBL_ERR_BITS;
  if (!(eps > 0.0f) || !isfinite(eps)) return HBL_ERR_EPS;
  if (seq_len < 0 || (bos_codes != nullptr && seq_len == 0)) return HBL_ERR_SHAPE;
  if (tokens == 0) return HBL_OK;
  if (!x || !codes || !scale) return HBL_ERR_NULL;
  if (bos_codes != nullptr && !bos_scale) return HBL_ERR_NULL;
  if (!aligned(x, 16) || !aligned(codes, 16) || !aligned(scale, 4) || !aligned(bos_codes, 16) || !aligned(bos_scale, 4))
    return HBL_ERR_ALIGN;
  return launch_kv_quant(x, (long)tokens * n_heads, n_heads, head_dim, bits, seq_len, eps, codes, scale, bos_codes, bos_scale,
                         static_cast<cudaStream_t>(stream));
}

int hbl_unpack_weights(const void* W_packed, int out_dim, int in_dim, int8_t* w_out, void* stream) {
  int rc = check_dims(0, in_dim, out_dim);
  if (rc != HBL_OK) return rc;
  if (!W_packed || !w_out) return HBL_ERR_NULL;
  if (!aligned(W_packed, 16) || !aligned(w_out, 16)) return HBL_ERR_ALIGN;
  return launch_unpack_weights(W_packed, out_dim, in_dim, w_out, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
