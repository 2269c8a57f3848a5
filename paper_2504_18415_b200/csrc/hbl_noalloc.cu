// hbl_gemm_i32_static: the streaming contraction kernel for callers that cannot
// provide (or allocate) a workspace.  Its scratch -- the slots in which CTAs hand
// partial sums of a shared row block to the block's owner, and the flags that say
// a slot is complete -- lives in a fixed array inside the library's device image
// instead of in caller memory.
#include "hbl_common.cuh"

using namespace hbl;

namespace {

constexpr int kStaticMaxTokens = 16;
constexpr size_t kStaticAccWords = 160 * 128 * kStaticMaxTokens;   // one 128-row x 16-token slot of partial sums per CTA (1.25 MiB)
constexpr size_t kStaticCounterWords = 1024;         // the contraction's flag words (one per CTA and pass)
constexpr size_t kStaticScratchBytes = (kStaticAccWords + kStaticCounterWords) * sizeof(int32_t);

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` only names the symbol; its device address is
// looked up once per device, with that device current.
int static_scratch_address(unsigned char** out) {
  static unsigned char* cached[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HBL_ERR_CUDA;
  if (cached[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return HBL_ERR_CUDA;
    cached[dev] = static_cast<unsigned char*>(p);
  }
  *out = cached[dev];
  return HBL_OK;
}

}  // namespace

extern "C" int hbl_gemm_i32_static(const int8_t* codes, const int32_t* codesum, int tokens, int in_dim,
                                   const void* W_packed, int out_dim, int32_t* acc_out, void* stream) {
  if (tokens < 0 || in_dim <= 0 || out_dim <= 0) return HBL_ERR_SHAPE;
  if (in_dim % 128 != 0 || out_dim % 16 != 0) return HBL_ERR_SHAPE;
  if (tokens > kStaticMaxTokens || in_dim > 32768) return HBL_ERR_TOO_LARGE;
  const size_t acc_words = gemm_stream_acc_words(tokens, out_dim);
  const size_t counter_words = gemm_stream_counter_words(out_dim);
  if (acc_words > kStaticAccWords || counter_words > kStaticCounterWords) return HBL_ERR_TOO_LARGE;   // cannot happen within the token limit
  if (tokens == 0) return HBL_OK;
  if (!codes || !codesum || !W_packed || !acc_out) return HBL_ERR_NULL;
  if (!aligned(codes, 16) || !aligned(W_packed, 16) || !aligned(acc_out, 16)) return HBL_ERR_ALIGN;
  unsigned char* scratch = nullptr;
  int rc = static_scratch_address(&scratch);
  if (rc != HBL_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int* counters = reinterpret_cast<int*>(scratch);
  int32_t* acc_ws = reinterpret_cast<int32_t*>(scratch + kStaticCounterWords * sizeof(int32_t));
  // The array keeps the previous call's contents.  Only the ready flags must be zero when the kernel
  // starts; a partial-sum slot is written in full by its thread block before its flag is raised, so
  // what an earlier call left there is never read.
  HBL_CUDA_OK(cudaMemsetAsync(counters, 0, counter_words * sizeof(int), s));
  return launch_gemm_stream(codes, nullptr, codesum, tokens, in_dim, W_packed, out_dim, nullptr, nullptr, acc_out,
                            acc_ws, counters, s);
}
