// Small-batch contraction of H-BitLinear (Eq. 7), weight-streaming bound.
//
// At T <= 64 tokens every packed weight byte is used once and the call is bound
// by how fast the 2-bit weights stream out of HBM.  Each warp reads its weight
// tiles with 128-bit loads straight into registers (the packed format is the
// register fragment order of the m16n8k32 integer MMA, see hbl_weights.cu),
// widens 16 weights with four shift-and-mask operations and contracts them with
// the tokens' int8 codes, which the CTA stages once in shared memory.  Nothing
// but the packed bytes crosses shared memory or HBM on the weight side.
//
// Weights are stored as u = w + 1 and fed as unsigned bytes, so the MMA computes
// sum_k u*q = sum_k w*q + sum_k q; the per-token code sum is subtracted in the
// epilogue (exact in int32).
//
// A CTA owns 128 weight rows x Kc columns.  When K is split over several CTAs
// the partial sums are combined with integer atomics (associative, so the
// result does not depend on arrival order) into a zeroed scratch array and the
// last CTA to arrive for a row group runs the epilogue.
#include "hbl_common.cuh"

namespace hbl {
namespace {

constexpr int kWarps = 4;
constexpr int kSlabsPerWarp = 2;
constexpr int kRowsPerCta = kWarps * kSlabsPerWarp * 16;   // 128
constexpr int kDepth = 4;                                  // k-blocks of weights in flight per lane

__device__ __forceinline__ void mma_u8s8(int (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// NT = number of 8-token MMA tiles (padded tokens = 8*NT).
template <int NT>
__global__ void __launch_bounds__(kWarps * 32)
gemm_stream_kernel(const int8_t* __restrict__ codes, const float* __restrict__ scale,
                   const int32_t* __restrict__ codesum, int T, int K, int Kc,
                   const uint4* __restrict__ Wp, int N, const float* __restrict__ alpha,
                   __nv_bfloat16* __restrict__ y, int32_t* __restrict__ acc_out,
                   int32_t* __restrict__ acc_ws, int* __restrict__ counters) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ int s_is_last;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const int splits = K / Kc;
  const int rg = blockIdx.x / splits;            // row group
  const int sp = blockIdx.x % splits;            // k split
  const int k0 = sp * Kc;
  const int ctiles = K / 128;
  const int nkb = Kc / 128;
  const int stride = Kc + 16;                    // bytes per staged token row
  constexpr int TP = 8 * NT;

  // ---- start the weight stream before anything else ----
  const int rt0 = rg * (kRowsPerCta / 16) + warp * kSlabsPerWarp;
  const int n_rt = N / 16;
  const uint4* wsrc[kSlabsPerWarp];
  bool slab_ok[kSlabsPerWarp];
#pragma unroll
  for (int s = 0; s < kSlabsPerWarp; ++s) {
    slab_ok[s] = (rt0 + s) < n_rt;
    wsrc[s] = Wp + ((size_t)(slab_ok[s] ? rt0 + s : 0) * ctiles + k0 / 128) * 32 + lane;
  }
  uint4 ring[kDepth][kSlabsPerWarp];
#pragma unroll
  for (int d = 0; d < kDepth; ++d)
#pragma unroll
    for (int s = 0; s < kSlabsPerWarp; ++s)
      ring[d][s] = (d < nkb && slab_ok[s]) ? __ldcs(wsrc[s] + (size_t)d * 32) : make_uint4(0, 0, 0, 0);

  // ---- stage this CTA's slice of the codes: [TP][Kc] bytes, rows >= T zero ----
  {
    const int vec_per_row = Kc / 16;
    for (int i = tid; i < TP * vec_per_row; i += kWarps * 32) {
      const int r = i / vec_per_row, c = i % vec_per_row;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (r < T) v = *reinterpret_cast<const uint4*>(codes + (size_t)r * K + k0 + c * 16);
      *reinterpret_cast<uint4*>(smem_raw + (size_t)r * stride + c * 16) = v;
    }
  }
  __syncthreads();

  int acc[kSlabsPerWarp][NT][4];
#pragma unroll
  for (int s = 0; s < kSlabsPerWarp; ++s)
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[s][n][i] = 0;

  const unsigned char* brow = smem_raw + (size_t)g * stride + 4 * t4;
  for (int kb0 = 0; kb0 < nkb; kb0 += kDepth) {
#pragma unroll
    for (int d = 0; d < kDepth; ++d) {
      const int kb = kb0 + d;
      if (kb < nkb) {
        uint4 cur[kSlabsPerWarp];
#pragma unroll
        for (int s = 0; s < kSlabsPerWarp; ++s) {
          cur[s] = ring[d][s];
          if (kb + kDepth < nkb && slab_ok[s]) ring[d][s] = __ldcs(wsrc[s] + (size_t)(kb + kDepth) * 32);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint32_t b0[NT], b1[NT];
#pragma unroll
          for (int n = 0; n < NT; ++n) {
            const unsigned char* p = brow + (size_t)n * 8 * stride + kb * 128 + j * 32;
            b0[n] = *reinterpret_cast<const uint32_t*>(p);
            b1[n] = *reinterpret_cast<const uint32_t*>(p + 16);
          }
#pragma unroll
          for (int s = 0; s < kSlabsPerWarp; ++s) {
            const uint32_t w = (j == 0) ? cur[s].x : (j == 1) ? cur[s].y : (j == 2) ? cur[s].z : cur[s].w;
            uint32_t a[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = (w >> (2 * i)) & 0x03030303u;
#pragma unroll
            for (int n = 0; n < NT; ++n) mma_u8s8(acc[s][n], a, b0[n], b1[n]);
          }
        }
      }
    }
  }

  // ---- combine / epilogue ----
  // Fragment element i of acc[s][n]: weight row rbase + g + 8*(i>>1), token 8n + 2*t4 + (i&1).
  const bool direct = (splits == 1);
  if (direct) {
    const float al = (acc_out == nullptr) ? __ldg(alpha) : 0.f;
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int tok = 8 * n + 2 * t4 + (i & 1);
        if (tok >= T) continue;
        const int cs = __ldg(codesum + tok);
        const float f = (acc_out == nullptr) ? __ldg(scale + tok) * al : 0.f;
#pragma unroll
        for (int s = 0; s < kSlabsPerWarp; ++s) {
          if (!slab_ok[s]) continue;
          const int row = (rt0 + s) * 16 + g + 8 * (i >> 1);
          const int a = acc[s][n][i] - cs;
          if (acc_out != nullptr) acc_out[(size_t)tok * N + row] = a;
          else y[(size_t)tok * N + row] = __float2bfloat16_rn((float)a * f);
        }
      }
    return;
  }
#pragma unroll
  for (int n = 0; n < NT; ++n)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int tok = 8 * n + 2 * t4 + (i & 1);
      if (tok >= T) continue;
#pragma unroll
      for (int s = 0; s < kSlabsPerWarp; ++s) {
        if (!slab_ok[s]) continue;
        const int row = (rt0 + s) * 16 + g + 8 * (i >> 1);
        atomicAdd(acc_ws + (size_t)tok * N + row, acc[s][n][i]);
      }
    }
  __threadfence();
  __syncthreads();
  if (tid == 0) s_is_last = (atomicAdd(counters + rg, 1) == splits - 1);
  __syncthreads();
  if (!s_is_last) return;
  __threadfence();
  {
    const float al = (acc_out == nullptr) ? __ldg(alpha) : 0.f;
    const int row_base = rg * kRowsPerCta;
    const int rows = min(kRowsPerCta, N - row_base);
    for (int i = tid; i < T * rows; i += kWarps * 32) {
      const int tok = i / rows, row = row_base + i % rows;
      const int a = __ldcg(acc_ws + (size_t)tok * N + row) - __ldg(codesum + tok);
      if (acc_out != nullptr) acc_out[(size_t)tok * N + row] = a;
      else y[(size_t)tok * N + row] = __float2bfloat16_rn((float)a * (__ldg(scale + tok) * al));
    }
  }
}

int choose_kc(int N, int K, int max_kc) {
  const int row_groups = (N + kRowsPerCta - 1) / kRowsPerCta;
  const int cands[5] = {2048, 1024, 512, 256, 128};
  int smallest = 128;
  for (int i = 0; i < 5; ++i) {
    if (cands[i] > max_kc || K % cands[i] != 0) continue;
    smallest = cands[i];
    if ((long)row_groups * (K / cands[i]) >= 148L * 3) return cands[i];
  }
  return smallest;
}

template <int NT>
int launch_nt(const int8_t* codes, const float* scale, const int32_t* codesum, int T, int K,
              const void* Wp, int N, const float* alpha, __nv_bfloat16* y, int32_t* acc_out,
              int32_t* acc_ws, int* counters, cudaStream_t s) {
  const int Kc = choose_kc(N, K, NT <= 2 ? 2048 : (NT == 4 ? 1024 : 512));   // staged codes stay <= 33 KiB
  const int splits = K / Kc;
  const int row_groups = (N + kRowsPerCta - 1) / kRowsPerCta;
  const size_t smem = (size_t)8 * NT * (Kc + 16);
  auto kern = gemm_stream_kernel<NT>;
  profile_before(KERNEL_CONTRACT, s);
  kern<<<row_groups * splits, kWarps * 32, smem, s>>>(codes, scale, codesum, T, K, Kc,
                                                      static_cast<const uint4*>(Wp), N, alpha, y, acc_out,
                                                      acc_ws, counters);
  profile_after(KERNEL_CONTRACT, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

}  // namespace

size_t gemm_stream_acc_words(int T, int N) { return (size_t)T * N; }
size_t gemm_stream_counter_words(int N) { return (size_t)(N + kRowsPerCta - 1) / kRowsPerCta; }

// acc_ws [T*N] and counters must be zero on entry when K is split (the caller
// clears them; the activation kernel does it as a side job in hbl_forward).
int launch_gemm_stream(const int8_t* codes, const float* scale, const int32_t* codesum, int T, int K,
                       const void* W_packed, int N, const float* alpha, __nv_bfloat16* y,
                       int32_t* acc_out, int32_t* acc_ws, int* counters, cudaStream_t s) {
  if (T <= 0) return HBL_OK;
  if (T > 64) return HBL_ERR_TOO_LARGE;
  if (T <= 8) return launch_nt<1>(codes, scale, codesum, T, K, W_packed, N, alpha, y, acc_out, acc_ws, counters, s);
  if (T <= 16) return launch_nt<2>(codes, scale, codesum, T, K, W_packed, N, alpha, y, acc_out, acc_ws, counters, s);
  if (T <= 32) return launch_nt<4>(codes, scale, codesum, T, K, W_packed, N, alpha, y, acc_out, acc_ws, counters, s);
  return launch_nt<8>(codes, scale, codesum, T, K, W_packed, N, alpha, y, acc_out, acc_ws, counters, s);
}

}  // namespace hbl
