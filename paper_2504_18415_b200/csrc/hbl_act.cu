// Activation side of the H-BitLinear forward pass: the Walsh-Hadamard transform
// of each token (Eq. 3-4), the per-token statistic and the INT8 / INT4 quantizer
// (Eq. 5-6), fused in one kernel.  One group of K/E threads owns one token and
// keeps its E = 32 or 64 elements per thread in registers for the whole pass.
//
// The transform H_m = H_2 (x) ... (x) H_2 acts on the m index bits independently,
// so its butterfly stages commute.  Each "phase" makes a set of index bits
// thread-local (a register layout), runs those stages in registers, and hands
// the vector to the next layout through shared memory:
//   phase 0  bits {0,1,2} and the top e-3 bits: what a coalesced 128-bit load gives;
//   phase 1  bits [3, 3+e) (only when m is large enough to need it);
//   final    the bits still missing, placed so that each thread also holds a
//            run of >= 4 consecutive indices: codes are packed in registers
//            and stored straight to global memory, coalesced.
// The shared-memory word address is XOR-swizzled so that the vector stores of
// phase 0, the scalar accesses of phase 1 and the vector loads of the final
// phase are all bank-conflict free.
#include <type_traits>

#include "hbl_common.cuh"
#include "hbl_quant_rows.cuh"

namespace hbl {

namespace {

// ---- register layouts ---------------------------------------------------------
// Local index j (e bits): its low NA bits sit at index bits [LOA, LOA+NA), the
// remaining NB bits at [LOB, LOB+NB).  Thread-id bits fill the other positions
// in increasing order.
template <int LOA, int NA, int LOB, int NB>
struct Layout {
  __host__ __device__ static constexpr int off(int j) {
    return ((j & ((1 << NA) - 1)) << LOA) | ((NB > 0) ? ((j >> NA) << LOB) : 0);
  }
  __device__ static int base(int tid) {
    int t0 = tid & ((1 << LOA) - 1);
    int r = tid >> LOA;
    if constexpr (NB == 0) {
      return t0 | (r << (LOA + NA));
    } else {
      constexpr int gap = LOB - (LOA + NA);
      int t1 = r & ((1 << gap) - 1);
      int t2 = r >> gap;
      return t0 | (t1 << (LOA + NA)) | (t2 << (LOB + NB));
    }
  }
};

// GF(2)-linear swizzle of the word address inside one token's buffer.
__host__ __device__ constexpr int swz(int a) {
  return a ^ ((a >> 3) & 0x1C) ^ ((a >> 5) & 0x18) ^ ((a >> 7) & 0x08);
}

template <int M, int E>
struct Plan {
  static constexpr int e = ilog2(E);
  static constexpr int R = M - e;                       // bits left after phase 0
  static constexpr bool two_mid = (R > e - 2);          // needs the middle phase
  using L0 = Layout<0, 3, M - (e - 3), e - 3>;
  using L1 = Layout<3, e, 0, 0>;                        // bits [3, 3+e)
  // final phase: r new bits starting at lo_n, plus e-r old low bits for contiguity
  static constexpr int lo_n = two_mid ? 3 + e : 3;
  static constexpr int r = two_mid ? (M - 2 * e) : R;
  static constexpr bool contiguous = (e - r >= lo_n);   // field collapses to [0, e)
  using LF = typename std::conditional<contiguous, Layout<0, e, 0, 0>,
                                       Layout<0, e - r, lo_n, r>>::type;
  static constexpr int new_lo = contiguous ? lo_n : (e - r);   // first new local bit
  static constexpr int run = contiguous ? E : (1 << (e - r));  // consecutive indices per thread
};

template <int E, int B0, int B1>
__device__ __forceinline__ void butterflies(float (&v)[E]) {
#pragma unroll
  for (int b = B0; b < B1; ++b) {
#pragma unroll
    for (int j = 0; j < E; ++j) {
      if ((j >> b) & 1) continue;
      float a = v[j], c = v[j | (1 << b)];
      v[j] = a + c;
      v[j | (1 << b)] = a - c;
    }
  }
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Reduce a float / int over the NT threads of one token group.  Fixed order.
template <int NT, bool IS_MAX>
__device__ __forceinline__ float group_reduce(float v, float* red, int group_warp0, int lane, int warp,
                                              int tid) {
  constexpr int W = (NT < 32) ? NT : 32;
#pragma unroll
  for (int o = W / 2; o > 0; o >>= 1) {
    float u = __shfl_xor_sync(0xffffffffu, v, o);
    v = IS_MAX ? fmaxf(v, u) : (v + u);
  }
  if (NT > 32) {
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = red[group_warp0];
#pragma unroll 1
    for (int w = 1; w < NT / 32; ++w) {
      float u = red[group_warp0 + w];
      t = IS_MAX ? fmaxf(t, u) : (t + u);
    }
    v = t;
  }
  return v;
}

constexpr float kSqrt7 = 2.6457513110645906f;
constexpr float kMagicRound = 12582912.0f;          // 1.5 * 2^23: y + kMagicRound has rint(y) in its low mantissa bits

// Four products -> four codes in one word: clamp, then round by the magic-number add (exact for |y| < 2^22, ties
// to even; no float-to-int conversion, which issues at a quarter of the rate).  The same decisions as
// clamp(rint(y)) for every finite y.
__device__ __forceinline__ uint32_t codes4(float y0, float y1, float y2, float y3, float lo, float hi) {
  const uint32_t a = __float_as_uint(fminf(fmaxf(y0, lo), hi) + kMagicRound), b = __float_as_uint(fminf(fmaxf(y1, lo), hi) + kMagicRound);
  const uint32_t c = __float_as_uint(fminf(fmaxf(y2, lo), hi) + kMagicRound), d = __float_as_uint(fminf(fmaxf(y3, lo), hi) + kMagicRound);
  return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}

// One CTA = TPC token groups of NT = K/E threads.
template <int M, int E, bool HAD>
__global__ void __launch_bounds__((((1 << M) / E) < 128 ? 128 : ((1 << M) / E)))
act_quant_kernel(const void* __restrict__ xin, int x_is_bf16, int T, int bits, float eps,
                 int8_t* __restrict__ codes, float* __restrict__ scale, int32_t* __restrict__ codesum,
                 float* __restrict__ xr_out, int32_t* __restrict__ zero_fill, size_t zero_words) {
  constexpr int K = 1 << M;
  constexpr int NT = K / E;
  constexpr int THREADS = NT < 128 ? 128 : NT;
  constexpr int TPC = THREADS / NT;
  constexpr int PAD = (NT < 32) ? NT : 0;
  using P = Plan<M, E>;
  using L0 = typename P::L0;
  using L1 = typename P::L1;
  using LF = typename P::LF;

  extern __shared__ __align__(16) float smem[];
  __shared__ float red_f[32];
  __shared__ int red_i[TPC];

  grid_launch_dependents();   // a programmatic dependent may start; it waits before reading our output
  const int tid_cta = threadIdx.x;
  // side job: clear the caller's scratch words (split-K accumulators of the next kernel)
  if (zero_fill != nullptr) {
    size_t n = zero_words;
    for (size_t i = (size_t)blockIdx.x * THREADS + tid_cta; i < n; i += (size_t)gridDim.x * THREADS)
      zero_fill[i] = 0;
  }

  const int g = tid_cta / NT;             // token group inside the CTA
  const int tid = tid_cta % NT;           // thread inside the group
  const int lane = tid_cta & 31, warp = tid_cta >> 5;
  const int group_warp0 = (NT >= 32) ? g * (NT / 32) : 0;
  const long token = (long)blockIdx.x * TPC + g;
  const bool live = token < T;
  float* buf = smem + g * (K + PAD);
  if (tid_cta < TPC) red_i[tid_cta] = 0;

  float v[E];
  // ---- phase 0: coalesced load, 8 consecutive elements per (thread, jB) ----
  {
    const int b0 = L0::base(tid);
    constexpr int NV = E / 8;
#pragma unroll
    for (int jb = 0; jb < NV; ++jb) {
      const long idx = token * K + b0 + L0::off(jb * 8);
      if (!live) {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[jb * 8 + i] = 0.f;
      } else if (x_is_bf16) {
        uint4 w = __ldg(reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(xin) + idx));
        v[jb * 8 + 0] = bf16_lo(w.x); v[jb * 8 + 1] = bf16_hi(w.x);
        v[jb * 8 + 2] = bf16_lo(w.y); v[jb * 8 + 3] = bf16_hi(w.y);
        v[jb * 8 + 4] = bf16_lo(w.z); v[jb * 8 + 5] = bf16_hi(w.z);
        v[jb * 8 + 6] = bf16_lo(w.w); v[jb * 8 + 7] = bf16_hi(w.w);
      } else {
        const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(xin) + idx);
        float4 a = __ldg(p), c = __ldg(p + 1);
        v[jb * 8 + 0] = a.x; v[jb * 8 + 1] = a.y; v[jb * 8 + 2] = a.z; v[jb * 8 + 3] = a.w;
        v[jb * 8 + 4] = c.x; v[jb * 8 + 5] = c.y; v[jb * 8 + 6] = c.z; v[jb * 8 + 7] = c.w;
      }
    }
  }

  if (HAD) {
    butterflies<E, 0, P::e>(v);
    // ---- exchange 0 -> (1 | final) ----
    {
      const int sb = swz(L0::base(tid));
#pragma unroll
      for (int j = 0; j < E; j += 4) {
        float4 q = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        *reinterpret_cast<float4*>(buf + (sb ^ swz(L0::off(j)))) = q;
      }
    }
    __syncthreads();
    if (P::two_mid) {
      const int sb = swz(L1::base(tid));
#pragma unroll
      for (int j = 0; j < E; ++j) v[j] = buf[sb ^ swz(L1::off(j))];
      butterflies<E, 0, P::e>(v);
#pragma unroll
      for (int j = 0; j < E; ++j) buf[sb ^ swz(L1::off(j))] = v[j];
      __syncthreads();
    }
    {
      const int sb = swz(LF::base(tid));
#pragma unroll
      for (int j = 0; j < E; j += 4) {
        float4 q = *reinterpret_cast<const float4*>(buf + (sb ^ swz(LF::off(j))));
        v[j] = q.x; v[j + 1] = q.y; v[j + 2] = q.z; v[j + 3] = q.w;
      }
      butterflies<E, P::new_lo, P::new_lo + P::r>(v);
    }
  }
  // Register layout from here on: LF when transformed, L0 otherwise.
  constexpr int RUN = HAD ? P::run : 8;
  const int obase = HAD ? LF::base(tid) : L0::base(tid);

  const float norm = HAD ? rsqrtf((float)K) : 1.0f;   // exact for K = 4^i, else 1 ulp
  if (xr_out != nullptr) {
    if (live) {
#pragma unroll
      for (int j = 0; j < E; j += 4) {
        const int o = HAD ? LF::off(j) : L0::off(j);
        float4 q = make_float4(v[j] * norm, v[j + 1] * norm, v[j + 2] * norm, v[j + 3] * norm);
        *reinterpret_cast<float4*>(xr_out + token * K + obase + o) = q;
      }
    }
    return;   // uniform over the grid: stage export only
  }

  // ---- per-token statistic (Eq. 5: max|x_r|; Eq. 6: mean|x_r|) ----
  float st;
  if (bits == 8) {
    float m = 0.f;
#pragma unroll
    for (int j = 0; j < E; ++j) m = fmaxf(m, fabsf(v[j]));
    m = group_reduce<NT, true>(m, red_f, group_warp0, lane, warp, tid);
    st = m * norm;
  } else {
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int j = 0; j < E; j += 4) {
      s0 += fabsf(v[j]); s1 += fabsf(v[j + 1]); s2 += fabsf(v[j + 2]); s3 += fabsf(v[j + 3]);
    }
    float s = group_reduce<NT, false>((s0 + s1) + (s2 + s3), red_f, group_warp0, lane, warp, tid);
    st = (s * norm) * (1.0f / (float)K);   // K is a power of two: exact scaling
  }
  const float c = (bits == 8) ? 127.0f : kSqrt7;
  const float rq = __fdiv_rn(c, st + eps) * norm;
  const float lo = (bits == 8) ? -128.0f : -8.0f, hi = (bits == 8) ? 127.0f : 7.0f;

  // ---- quantize, pack 4 codes per word, store runs of RUN consecutive codes ----
  int csum = 0;
#pragma unroll
  for (int j0 = 0; j0 < E; j0 += RUN) {
    uint32_t words[RUN / 4];
#pragma unroll
    for (int w = 0; w < RUN / 4; ++w) {
      const int j = j0 + w * 4;
      words[w] = codes4(v[j] * rq, v[j + 1] * rq, v[j + 2] * rq, v[j + 3] * rq, lo, hi);
      csum = __dp4a((int)words[w], 0x01010101, csum);
    }
    if (live) {
      const int o = HAD ? LF::off(j0) : L0::off(j0);
      int8_t* dst = codes + token * K + obase + o;
      if (RUN >= 16) {
#pragma unroll
        for (int w = 0; w < RUN / 4; w += 4)
          *reinterpret_cast<uint4*>(dst + 4 * w) = make_uint4(words[w], words[w + 1], words[w + 2], words[w + 3]);
      } else if (RUN == 8) {
        *reinterpret_cast<uint2*>(dst) = make_uint2(words[0], words[1]);
      } else {
        *reinterpret_cast<uint32_t*>(dst) = words[0];
      }
    }
  }
  // ---- code sum and scale ----
#pragma unroll
  for (int o = ((NT < 32) ? NT : 32) / 2; o > 0; o >>= 1) csum += __shfl_xor_sync(0xffffffffu, csum, o);
  if (NT > 32) {
    __syncthreads();   // red_i was cleared before the first barrier of group_reduce
    if (lane == 0) atomicAdd(&red_i[g], csum);
    __syncthreads();
    csum = red_i[g];
  }
  if (live && tid == 0) {
    scale[token] = __fdiv_rn(st, c);
    if (codesum != nullptr) codesum[token] = csum;
  }
  grid_dependency_wait();   // chain: this kernel is complete only when the one before it is
}

// No transform and K not a power of two: a plain two-pass kernel, one CTA per
// token; pass 2 re-reads the token (it is still in L1/L2).
__global__ void __launch_bounds__(256)
act_quant_generic_kernel(const void* __restrict__ xin, int x_is_bf16, int T, int K, int bits, float eps,
                         int8_t* __restrict__ codes, float* __restrict__ scale,
                         int32_t* __restrict__ codesum, int32_t* __restrict__ zero_fill,
                         size_t zero_words) {
  __shared__ float red_f[8];
  __shared__ int red_i[8];
  grid_launch_dependents();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (zero_fill != nullptr)
    for (size_t i = (size_t)blockIdx.x * 256 + tid; i < zero_words; i += (size_t)gridDim.x * 256)
      zero_fill[i] = 0;
  const long token = blockIdx.x;
  auto load4 = [&](int k, float (&f)[4]) {
    if (x_is_bf16) {
      uint2 w = *reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(xin) + token * K + k);
      f[0] = bf16_lo(w.x); f[1] = bf16_hi(w.x); f[2] = bf16_lo(w.y); f[3] = bf16_hi(w.y);
    } else {
      float4 a = *reinterpret_cast<const float4*>(static_cast<const float*>(xin) + token * K + k);
      f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w;
    }
  };
  float acc = 0.f;
  for (int k = tid * 4; k < K; k += 1024) {
    float f[4];
    load4(k, f);
    if (bits == 8) acc = fmaxf(acc, fmaxf(fmaxf(fabsf(f[0]), fabsf(f[1])), fmaxf(fabsf(f[2]), fabsf(f[3]))));
    else acc += (fabsf(f[0]) + fabsf(f[1])) + (fabsf(f[2]) + fabsf(f[3]));
  }
  for (int o = 16; o > 0; o >>= 1) {
    float u = __shfl_xor_sync(0xffffffffu, acc, o);
    acc = (bits == 8) ? fmaxf(acc, u) : acc + u;
  }
  if (lane == 0) red_f[warp] = acc;
  __syncthreads();
  float st = red_f[0];
  for (int w = 1; w < 8; ++w) st = (bits == 8) ? fmaxf(st, red_f[w]) : st + red_f[w];
  if (bits != 8) st = st / (float)K;
  const float c = (bits == 8) ? 127.0f : kSqrt7;
  const float rq = __fdiv_rn(c, st + eps);
  const float lo = (bits == 8) ? -128.0f : -8.0f, hi = (bits == 8) ? 127.0f : 7.0f;
  int csum = 0;
  for (int k = tid * 4; k < K; k += 1024) {
    float f[4];
    load4(k, f);
    const uint32_t pk = codes4(f[0] * rq, f[1] * rq, f[2] * rq, f[3] * rq, lo, hi);
    csum = __dp4a((int)pk, 0x01010101, csum);
    *reinterpret_cast<uint32_t*>(codes + token * K + k) = pk;
  }
  for (int o = 16; o > 0; o >>= 1) csum += __shfl_xor_sync(0xffffffffu, csum, o);
  if (lane == 0) red_i[warp] = csum;
  __syncthreads();
  if (tid == 0) {
    int t = 0;
    for (int w = 0; w < 8; ++w) t += red_i[w];
    scale[token] = __fdiv_rn(st, c);
    if (codesum != nullptr) codesum[token] = t;
  }
  grid_dependency_wait();
}

// bf16 input, no transform, any K that is a multiple of 128: the body is in hbl_quant_rows.cuh.
template <int BITS>
__global__ void __launch_bounds__(512, 2)
quant_rows_bf16_kernel(const __nv_bfloat16* __restrict__ x, int T, int K, int NT, float eps,
                       int8_t* __restrict__ codes, float* __restrict__ scale, int32_t* __restrict__ codesum,
                       int32_t* __restrict__ zero_fill, size_t zero_words, int packed) {
  __shared__ float red_f[16];
  __shared__ int red_i[16];
  grid_launch_dependents();   // a programmatic dependent may start; it waits before reading our output
  if (zero_fill != nullptr)
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < zero_words; i += (size_t)gridDim.x * blockDim.x)
      zero_fill[i] = 0;
  quant_rows_bf16_body<BITS>(x, T, K, NT, eps, codes, scale, codesum, packed, (long)blockIdx.x, red_f, red_i);
  grid_dependency_wait();   // chain: this kernel is complete only when the one before it is
}

int launch_quant_rows_bf16(const void* x, int T, int K, int bits, float eps, int8_t* codes, float* scale,
                           int32_t* codesum, int32_t* zf, size_t zw, cudaStream_t s, bool packed) {
  const int n_chunks = K / 8;
  const int NT = ((n_chunks + 7) / 8 + 31) / 32 * 32;               // eight chunks per thread, whole warps
  if (NT > 512) return HBL_ERR_SHAPE;
  const int TPC = NT >= 128 ? 1 : 128 / NT;
  const int grid = (T + TPC - 1) / TPC;
  profile_before(KERNEL_ACT, s);
  if (bits == 8)
    HBL_CUDA_OK(launch_dependent(quant_rows_bf16_kernel<8>, dim3(grid), dim3(NT * TPC), 0, s,
                                 static_cast<const __nv_bfloat16*>(x), T, K, NT, eps, codes, scale, codesum, zf, zw, (int)packed));
  else
    HBL_CUDA_OK(launch_dependent(quant_rows_bf16_kernel<4>, dim3(grid), dim3(NT * TPC), 0, s,
                                 static_cast<const __nv_bfloat16*>(x), T, K, NT, eps, codes, scale, codesum, zf, zw, (int)packed));
  profile_after(KERNEL_ACT, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

template <int M, int E, bool HAD>
int launch_one(const void* x, int x_dtype, int T, int bits, float eps, int8_t* codes, float* scale,
               int32_t* codesum, float* xr_out, int32_t* zf, size_t zw, cudaStream_t s) {
  constexpr int K = 1 << M;
  constexpr int NT = K / E;
  constexpr int THREADS = NT < 128 ? 128 : NT;
  constexpr int TPC = THREADS / NT;
  constexpr int PAD = (NT < 32) ? NT : 0;
  const size_t smem = HAD ? sizeof(float) * TPC * (K + PAD) : 0;
  auto kern = act_quant_kernel<M, E, HAD>;
  if (smem > 48 * 1024) HBL_ALLOW_DYNAMIC_SMEM(kern, smem);
  const int grid = (T + TPC - 1) / TPC;
  profile_before(KERNEL_ACT, s);
  HBL_CUDA_OK(launch_dependent(kern, dim3(grid), dim3(THREADS), smem, s, x, (int)(x_dtype == HBL_BF16), T, bits, eps,
                               codes, scale, codesum, xr_out, zf, zw));
  profile_after(KERNEL_ACT, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

template <bool HAD>
int dispatch(int m, const void* x, int x_dtype, int T, int bits, float eps, int8_t* codes, float* scale,
             int32_t* codesum, float* xr_out, int32_t* zf, size_t zw, cudaStream_t s) {
#define HBL_CASE(MM, EE) \
  case MM: return launch_one<MM, EE, HAD>(x, x_dtype, T, bits, eps, codes, scale, codesum, xr_out, zf, zw, s);
  switch (m) {
    HBL_CASE(7, 32) HBL_CASE(8, 32) HBL_CASE(9, 64) HBL_CASE(10, 64) HBL_CASE(11, 32)
    HBL_CASE(12, 32) HBL_CASE(13, 32) HBL_CASE(14, 64) HBL_CASE(15, 64)
    default: return HBL_ERR_SHAPE;
  }
#undef HBL_CASE
}

}  // namespace

// Whether launch_act_quant can write INT4 codes two per byte for this call (the kernels that serve bf16 inputs
// can; the others write one code per byte).
bool act_quant_can_pack(int x_dtype, int T, int K, int bits, int use_hadamard) {
  if (bits != 4 || x_dtype != HBL_BF16) return false;
  if (use_hadamard) return act_quant_bf16_supported(K);
  return K % 128 == 0 && K <= 32768;
}

int launch_act_quant(const void* x, int x_dtype, int T, int K, int bits, int use_hadamard, float eps,
                     int8_t* codes, float* scale, int32_t* codesum, float* xr_out,
                     int32_t* zero_fill, size_t zero_fill_words, cudaStream_t s, bool packed) {
  if (T <= 0) return HBL_OK;
  if (packed && (xr_out != nullptr || !act_quant_can_pack(x_dtype, T, K, bits, use_hadamard))) return HBL_ERR_SHAPE;
  if (use_hadamard && x_dtype == HBL_BF16 && act_quant_bf16_supported(K))
    return launch_act_quant_bf16(x, T, K, bits, eps, codes, scale, codesum, xr_out, zero_fill, zero_fill_words, s, packed);
  if (!use_hadamard && x_dtype == HBL_BF16 && xr_out == nullptr && K % 128 == 0 && K <= 32768)
    return launch_quant_rows_bf16(x, T, K, bits, eps, codes, scale, codesum, zero_fill, zero_fill_words, s, packed);
  if (is_pow2(K)) {
    const int m = ilog2((unsigned)K);
    return use_hadamard
               ? dispatch<true>(m, x, x_dtype, T, bits, eps, codes, scale, codesum, xr_out, zero_fill, zero_fill_words, s)
               : dispatch<false>(m, x, x_dtype, T, bits, eps, codes, scale, codesum, xr_out, zero_fill, zero_fill_words, s);
  }
  if (use_hadamard) return HBL_ERR_NOT_POW2;
  if (xr_out != nullptr) return HBL_ERR_SHAPE;
  profile_before(KERNEL_ACT, s);
  HBL_CUDA_OK(launch_dependent(act_quant_generic_kernel, dim3(T), dim3(256), 0, s, x, (int)(x_dtype == HBL_BF16), T, K,
                               bits, eps, codes, scale, codesum, zero_fill, zero_fill_words));
  profile_after(KERNEL_ACT, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

}  // namespace hbl
