// Weight side of H-BitLinear: the per-tensor absmean ternary quantizer (Eq. 1-2)
// and the 2-bit storage format.
//
// Format (also described in hbl.h): W[N,K] is cut into tiles of 128 rows x 128
// columns (rows padded with zeros up to a multiple of 128), 4096 bytes each,
// ordered [row block][column block].  A tile is [h = 0,1][row 0..127][four 32-bit
// words]: word v of (h, row) holds the 16 weights of that row in columns
// 16*(4h+v) .. +15 of the tile, column 4*i + b at bit 8*b + 2*i, stored as
// u = w + 1 (0,1,2).  So (word >> 2*i) & 0x03030303 is four consecutive weights of
// one row as unsigned bytes -- what a thread that owns one row of a tensor-memory
// operand needs -- and a thread reads its row's 32 bytes with two conflict-free
// 128-bit shared-memory loads.
#include "hbl_common.cuh"

namespace hbl {
namespace {

constexpr int kReduceThreads = 256;
constexpr int kMaxPartials = 2048;

__device__ __forceinline__ float load_w(const void* W, int is_bf16, size_t i) {
  return is_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(W)[i]) : static_cast<const float*>(W)[i];
}

// Pass 1: fp64 partial sums of |W|, one per CTA, in a fixed order.
__global__ void __launch_bounds__(kReduceThreads)
absmean_partial_kernel(const void* __restrict__ W, int is_bf16, size_t total, double* __restrict__ partials) {
  __shared__ double red[kReduceThreads / 32];
  const size_t per_cta = (total / 4 + gridDim.x - 1) / gridDim.x;   // in groups of 4 elements
  const size_t g0 = (size_t)blockIdx.x * per_cta;
  const size_t g1 = min(g0 + per_cta, total / 4);
  double acc = 0.0;
  for (size_t g = g0 + threadIdx.x; g < g1; g += kReduceThreads) {
    float f0, f1, f2, f3;
    if (is_bf16) {
      uint2 w = reinterpret_cast<const uint2*>(W)[g];
      f0 = __uint_as_float(w.x << 16); f1 = __uint_as_float(w.x & 0xFFFF0000u);
      f2 = __uint_as_float(w.y << 16); f3 = __uint_as_float(w.y & 0xFFFF0000u);
    } else {
      float4 w = reinterpret_cast<const float4*>(W)[g];
      f0 = w.x; f1 = w.y; f2 = w.z; f3 = w.w;
    }
    acc += ((double)fabsf(f0) + (double)fabsf(f1)) + ((double)fabsf(f2) + (double)fabsf(f3));
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < kReduceThreads / 32; ++w) t += red[w];
    partials[blockIdx.x] = t;
  }
}

// Pass 2: every CTA re-derives alpha from the partials (fixed order), then
// ternarises and packs.  One thread = one packed word = 16 weights of one row.
__global__ void __launch_bounds__(256)
ternarise_pack_kernel(const void* __restrict__ W, int is_bf16, int N, int K, float eps,
                      const double* __restrict__ partials, int n_partials,
                      uint32_t* __restrict__ packed, float* __restrict__ alpha_out) {
  __shared__ float s_alpha;
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int i = 0; i < n_partials; ++i) t += partials[i];
    const float a = (float)(t / ((double)N * (double)K));
    s_alpha = a;
    if (blockIdx.x == 0) *alpha_out = a;
  }
  __syncthreads();
  const float d = s_alpha + eps;
  const int n_kb = K / 128;
  const size_t n_words = (size_t)((N + 127) / 128) * n_kb * 1024;
  for (size_t it = (size_t)blockIdx.x * 256 + threadIdx.x; it < n_words; it += (size_t)gridDim.x * 256) {
    const int v = (int)(it & 3), row = (int)((it >> 2) & 127), h = (int)((it >> 9) & 1);
    const size_t tile = it >> 10;
    const int kb = (int)(tile % n_kb), rb = (int)(tile / n_kb);
    const int R = rb * 128 + row;
    uint32_t wd = 0x55555555u;                                // padding rows: w = 0
    if (R < N) {
      wd = 0;
      const size_t base = (size_t)R * K + (size_t)kb * 128 + 16 * (4 * h + v);
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const float w = load_w(W, is_bf16, base + 4 * i + b);
          float r = rintf(__fdiv_rn(w, d));                 // round half to even
          r = fminf(fmaxf(r, -1.0f), 1.0f);
          wd |= (uint32_t)((int)r + 1) << (8 * b + 2 * i);
        }
    }
    packed[it] = wd;
  }
}

// Packed -> int8 [N,K] row-major (values -1,0,1).  One thread = one packed word = 16 weights of one row.
__global__ void __launch_bounds__(256)
unpack_kernel(const uint32_t* __restrict__ packed, int N, int K, int8_t* __restrict__ out) {
  const int n_kb = K / 128;
  const size_t n_words = (size_t)((N + 127) / 128) * n_kb * 1024;
  for (size_t it = (size_t)blockIdx.x * 256 + threadIdx.x; it < n_words; it += (size_t)gridDim.x * 256) {
    const int v = (int)(it & 3), row = (int)((it >> 2) & 127), h = (int)((it >> 9) & 1);
    const size_t tile = it >> 10;
    const int kb = (int)(tile % n_kb), rb = (int)(tile / n_kb);
    const int R = rb * 128 + row;
    if (R >= N) continue;
    const uint32_t wd = __ldg(packed + it);
    uint4 o;
    o.x = __vsub4(wd & 0x03030303u, 0x01010101u);            // per-byte w = u - 1: columns 0..3 of the 16
    o.y = __vsub4((wd >> 2) & 0x03030303u, 0x01010101u);
    o.z = __vsub4((wd >> 4) & 0x03030303u, 0x01010101u);
    o.w = __vsub4((wd >> 6) & 0x03030303u, 0x01010101u);
    *reinterpret_cast<uint4*>(out + (size_t)R * K + (size_t)kb * 128 + 16 * (4 * h + v)) = o;
  }
  // Launched as a programmatic dependent of the activation kernel (it reads nothing of it, so the two
  // overlap); completing only after that kernel keeps "unpack done" meaning "activations done" for
  // the contraction that follows.
  grid_dependency_wait();
}

}  // namespace

int launch_weight_quant(const void* W, int w_dtype, int N, int K, float eps, void* packed, float* alpha,
                        void* ws, cudaStream_t s) {
  const size_t total = (size_t)N * K;
  int grid = (int)min((size_t)kMaxPartials, (total / 4 + kReduceThreads * 8 - 1) / (kReduceThreads * 8));
  if (grid < 1) grid = 1;
  double* partials = static_cast<double*>(ws);
  absmean_partial_kernel<<<grid, kReduceThreads, 0, s>>>(W, w_dtype == HBL_BF16, total, partials);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  const size_t n_words = (size_t)((N + 127) / 128) * (K / 128) * 1024;
  int grid2 = (int)min((size_t)148 * 16, (n_words + 255) / 256);
  ternarise_pack_kernel<<<grid2, 256, 0, s>>>(W, w_dtype == HBL_BF16, N, K, eps, partials, grid,
                                              static_cast<uint32_t*>(packed), alpha);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

int launch_unpack_weights(const void* packed, int N, int K, int8_t* out, cudaStream_t s) {
  const size_t n_words = (size_t)((N + 127) / 128) * (K / 128) * 1024;
  int grid = (int)min((size_t)148 * 16, (n_words + 255) / 256);
  profile_before(KERNEL_UNPACK, s);
  HBL_CUDA_OK(launch_dependent(unpack_kernel, dim3(grid), dim3(256), 0, s, static_cast<const uint32_t*>(packed), N, K, out));
  profile_after(KERNEL_UNPACK, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

}  // namespace hbl
