// Weight side of H-BitLinear: the per-tensor absmean ternary quantizer (Eq. 1-2)
// and the 2-bit storage format.
//
// Format (also described in hbl.h): W[N,K] is cut into tiles of 16 rows x 128
// columns; a tile is 512 bytes = 32 "lanes" x four 32-bit words.  Word j of
// lane l carries the 16 weights that lane l of a warp feeds to one
// m16n8k32 integer MMA as its A fragment (four 8-bit x4 registers a0..a3):
//   a_i byte b  =  W[16*rt + (l>>2) + 8*(i&1)][128*ct + 32*j + 16*(i>>1) + 4*(l&3) + b]
// stored as u = w + 1 (0,1,2) at bit 8*b + 2*i, so that (word >> 2*i) & 0x03030303
// is register a_i, ready to use as four unsigned bytes.
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
// ternarises and packs.  One thread = one (tile, lane) = four packed words.
__global__ void __launch_bounds__(256)
ternarise_pack_kernel(const void* __restrict__ W, int is_bf16, int N, int K, float eps,
                      const double* __restrict__ partials, int n_partials,
                      uint4* __restrict__ packed, float* __restrict__ alpha_out) {
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
  const int ctiles = K / 128;
  const size_t n_items = (size_t)(N / 16) * ctiles * 32;
  for (size_t it = (size_t)blockIdx.x * 256 + threadIdx.x; it < n_items; it += (size_t)gridDim.x * 256) {
    const int l = (int)(it & 31);
    const size_t tile = it >> 5;
    const int ct = (int)(tile % ctiles);
    const int rt = (int)(tile / ctiles);
    const int row0 = rt * 16 + (l >> 2);
    const int col0 = ct * 128 + 4 * (l & 3);
    uint32_t words[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t wd = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const size_t base = (size_t)(row0 + 8 * (i & 1)) * K + col0 + 32 * j + 16 * (i >> 1);
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const float w = load_w(W, is_bf16, base + b);
          float r = rintf(__fdiv_rn(w, d));                 // round half to even
          r = fminf(fmaxf(r, -1.0f), 1.0f);
          wd |= (uint32_t)((int)r + 1) << (8 * b + 2 * i);
        }
      }
      words[j] = wd;
    }
    packed[it] = make_uint4(words[0], words[1], words[2], words[3]);
  }
}

// Packed -> int8 [N,K] row-major (values -1,0,1).  One thread = one (tile, lane).
__global__ void __launch_bounds__(256)
unpack_kernel(const uint4* __restrict__ packed, int N, int K, int8_t* __restrict__ out) {
  const int ctiles = K / 128;
  const size_t n_items = (size_t)(N / 16) * ctiles * 32;
  for (size_t it = (size_t)blockIdx.x * 256 + threadIdx.x; it < n_items; it += (size_t)gridDim.x * 256) {
    const int l = (int)(it & 31);
    const size_t tile = it >> 5;
    const int ct = (int)(tile % ctiles);
    const int rt = (int)(tile / ctiles);
    const int row0 = rt * 16 + (l >> 2);
    const int col0 = ct * 128 + 4 * (l & 3);
    const uint4 q = __ldg(packed + it);
    const uint32_t words[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t u = (words[j] >> (2 * i)) & 0x03030303u;   // four bytes in {0,1,2}
        const uint32_t s = __vsub4(u, 0x01010101u);               // per-byte w = u - 1
        const size_t base = (size_t)(row0 + 8 * (i & 1)) * K + col0 + 32 * j + 16 * (i >> 1);
        *reinterpret_cast<uint32_t*>(out + base) = s;
      }
    }
  }
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
  const size_t n_items = total / 16;
  int grid2 = (int)min((size_t)148 * 16, (n_items + 255) / 256);
  ternarise_pack_kernel<<<grid2, 256, 0, s>>>(W, w_dtype == HBL_BF16, N, K, eps, partials, grid,
                                              static_cast<uint4*>(packed), alpha);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

int launch_unpack_weights(const void* packed, int N, int K, int8_t* out, cudaStream_t s) {
  const size_t n_items = (size_t)N * K / 16;
  int grid = (int)min((size_t)148 * 16, (n_items + 255) / 256);
  profile_before(KERNEL_UNPACK, s);
  unpack_kernel<<<grid, 256, 0, s>>>(static_cast<const uint4*>(packed), N, K, out);
  profile_after(KERNEL_UNPACK, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

}  // namespace hbl
