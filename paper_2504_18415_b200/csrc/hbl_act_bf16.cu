// Activation side of H-BitLinear for bf16 inputs with the transform on: the
// Walsh-Hadamard transform of each token (Eq. 3-4), the per-token statistic and
// the INT8 / INT4 quantizer (Eq. 5-6) in one kernel, K = 2^M for M = 11..14.
//
// On this chip the transform is bound by instruction issue, not by HBM: at
// K = 8192 a token needs 13 butterfly stages per element while HBM delivers an
// element every ~0.4 ns per SM.  The kernel therefore spends as few issue slots
// per element as it can:
//
//   * The first four stages run on the tensor cores.  A 128-bit load gives a
//     lane eight consecutive bf16 values, which is exactly the A fragment of an
//     m16n8k16 MMA; multiplied by the 16x16 matrix of +-1 (exact in bf16, fp32
//     accumulation of exact products) two MMAs return the same eight positions
//     transformed over index bits {0,1,3,4} -- including the two bits that live
//     in other lanes, so no shuffle is needed -- and already widened to fp32.
//   * All other stages are packed fp32 butterflies (add/sub.f32x2: two
//     butterflies per issue slot) on 64 elements held in registers.
//   * One exchange through shared memory (XOR-swizzled, conflict free, 128-bit
//     stores) separates the two register layouts:
//       phase 0  index bits {0..4} and the top three bits (eight 16-byte chunks per lane);
//       final    the M-8 bits in between, plus the low 6-(M-8) bits for contiguity.
//   * Codes are assembled in shared memory (over the exchange buffer, which is
//     dead by then) and leave with coalesced 128-bit stores.
#include "hbl_common.cuh"

namespace hbl {
namespace {

constexpr float kSqrt7 = 2.6457513110645906f;
constexpr float kMagic = 12582912.0f;          // 1.5 * 2^23: x + kMagic has rint(x) in its low mantissa bits

// ---- packed fp32 pairs ---------------------------------------------------------
__device__ __forceinline__ void butterfly2(float2& a, float2& b) {
  float2 s, d;
  asm("{\n .reg .b64 ra, rb, rs, rd;\n mov.b64 ra, {%4, %5};\n mov.b64 rb, {%6, %7};\n"
      " add.rn.f32x2 rs, ra, rb;\n sub.rn.f32x2 rd, ra, rb;\n"
      " mov.b64 {%0, %1}, rs;\n mov.b64 {%2, %3}, rd;\n}"
      : "=f"(s.x), "=f"(s.y), "=f"(d.x), "=f"(d.y)
      : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
  a = s;
  b = d;
}

// Butterfly stages over bits [B0, B1) of the pair index (v holds 32 pairs).
template <int B0, int B1>
__device__ __forceinline__ void stages2(float2 (&v)[32]) {
#pragma unroll
  for (int b = B0; b < B1; ++b) {
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      if ((e >> b) & 1) continue;
      butterfly2(v[e], v[e | (1 << b)]);
    }
  }
}

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.0f));
}

// Word address swizzle of a token's exchange buffer: toggles bit 2 with bits 5 and 8,
// which keeps every 4-word vector intact and makes the phase-0 vector stores and the
// final-phase loads of every supported M bank-conflict free.
__device__ __forceinline__ int swz_word(int a) { return a ^ ((((a >> 5) ^ (a >> 8)) & 1) << 2); }
// Byte address swizzle of the code staging area (keeps 16-byte chunks intact).
__device__ __forceinline__ int swz_code(int i) { return i ^ (((i >> 9) & 3) << 5); }

template <int M>
struct Geometry {
  static constexpr int K = 1 << M;
  static constexpr int NT = K / 64;                       // threads per token
  static constexpr int THREADS = NT < 128 ? 128 : NT;
  static constexpr int TPC = THREADS / NT;                // tokens per CTA
  static constexpr int R = M - 8;                         // index bits [5, 5+R) are transformed in the final phase
  static constexpr int C = 6 - R;                         // low bits kept thread-local for contiguity
  static constexpr int RUN = 1 << C;                      // consecutive elements per thread in the final layout
  // 1/sqrt(K): exact for even M, one rounding otherwise
  static constexpr float NORM = (M % 2 == 0) ? 1.0f / (float)(1 << (M / 2))
                                             : 0.70710678118654752440f / (float)(1 << ((M - 1) / 2));
};

// Sum / max over the NT threads of one token group, in a fixed order.
template <int NT, bool IS_MAX>
__device__ __forceinline__ float group_reduce(float v, float* red, int group, int lane, int warp) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float u = __shfl_xor_sync(0xffffffffu, v, o);
    v = IS_MAX ? fmaxf(v, u) : (v + u);
  }
  if (NT > 32) {
    if (lane == 0) red[warp] = v;
    __syncthreads();
    constexpr int WPG = NT / 32;
    float t = red[group * WPG];
#pragma unroll
    for (int w = 1; w < WPG; ++w) {
      const float u = red[group * WPG + w];
      t = IS_MAX ? fmaxf(t, u) : (t + u);
    }
    v = t;
  } else {
    __syncthreads();   // every group reaches the same barriers
  }
  return v;
}

template <int M, int BITS>
__global__ void __launch_bounds__(Geometry<M>::THREADS, 512 / Geometry<M>::THREADS)
fwht_quant_bf16_kernel(const __nv_bfloat16* __restrict__ x, int T, float eps, int8_t* __restrict__ codes,
                       float* __restrict__ scale, int32_t* __restrict__ codesum, float* __restrict__ xr_out,
                       int32_t* __restrict__ zero_fill, size_t zero_words) {
  using G = Geometry<M>;
  constexpr int K = G::K, NT = G::NT, THREADS = G::THREADS, TPC = G::TPC, R = G::R, C = G::C, RUN = G::RUN;
  extern __shared__ __align__(16) float smem[];
  __shared__ float red_f[THREADS / 32];
  __shared__ int red_i[THREADS / 32];

  const int tid_cta = threadIdx.x;
  if (zero_fill != nullptr) {   // side job: clear the caller's scratch words
    for (size_t i = (size_t)blockIdx.x * THREADS + tid_cta; i < zero_words; i += (size_t)gridDim.x * THREADS)
      zero_fill[i] = 0;
  }
  const int group = tid_cta / NT;
  const int tid = tid_cta % NT;
  const int lane = tid_cta & 31, warp_cta = tid_cta >> 5;
  const int warp = tid >> 5;                               // warp inside the token group
  const long token = (long)blockIdx.x * TPC + group;
  const bool live = token < T;
  float* buf = smem + (size_t)group * K;

  // ---- the 16x16 sign matrix as B fragments (two MMAs: output columns 0-7 and 8-15) ----
  // k-bit domain of the MMA: k0 = index bit 0, k1 k2 = index bits 3 4 (the lane's t), k3 = index bit 1.
  uint32_t hb[2][2];
  {
    const int t = lane & 3, g = lane >> 2;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int n = g + 8 * j;
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int k_lo = 2 * t + 8 * r, k_hi = k_lo + 1;
        const uint32_t lo = (__popc(k_lo & n) & 1) ? 0xBF80u : 0x3F80u;
        const uint32_t hi = (__popc(k_hi & n) & 1) ? 0xBF80u : 0x3F80u;
        hb[j][r] = lo | (hi << 16);
      }
    }
  }

  // ---- phase 0: eight coalesced 16-byte chunks per lane; chunk c covers index
  //      c << (M-3) | warp << 8 | lane << 3 | m,  m = 0..7 ----
  float2 v[32];
  {
    const __nv_bfloat16* src = x + token * K + (warp << 8) + (lane << 3);
    uint4 raw[8];
#pragma unroll
    for (int c = 0; c < 8; ++c)
      raw[c] = live ? __ldg(reinterpret_cast<const uint4*>(src + ((size_t)c << (M - 3)))) : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      // A fragment: (x: m 0,1) rows g, k3 = 0; (z: m 4,5) rows g+8; (y: m 2,3) k3 = 1; (w: m 6,7) both
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        float d[4];
        mma_bf16_16816(d, raw[c].x, raw[c].z, raw[c].y, raw[c].w, hb[j][0], hb[j][1]);
        // d[2h + b] is position m = b + 2j + 4h; pair index p = j + 2h
        v[c * 4 + j] = make_float2(d[0], d[1]);
        v[c * 4 + j + 2] = make_float2(d[2], d[3]);
      }
    }
  }
  // pair index e = c*4 + p: bit 0 = index bit 1 (done), bit 1 = index bit 2, bits 2..4 = the chunk bits
  stages2<1, 5>(v);

  // ---- exchange ----
  {
    const int base = (warp << 8) | (lane << 3);
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const int a = swz_word(base | (c << (M - 3)));
      *reinterpret_cast<float4*>(buf + a) = make_float4(v[c * 4].x, v[c * 4].y, v[c * 4 + 1].x, v[c * 4 + 1].y);
      *reinterpret_cast<float4*>(buf + (a ^ 4)) = make_float4(v[c * 4 + 2].x, v[c * 4 + 2].y, v[c * 4 + 3].x, v[c * 4 + 3].y);
    }
  }
  __syncthreads();

  // ---- final layout: local j (6 bits): low C bits = index bits [0,C), high R bits = index bits [5,5+R) ----
  const int fbase = ((tid & ((1 << (5 - C)) - 1)) << C) | ((tid >> (5 - C)) << (M - 3));
  auto findex = [&](int j) { return fbase | (j & (RUN - 1)) | ((j >> C) << 5); };
#pragma unroll
  for (int jh = 0; jh < (1 << R); ++jh) {
    const int a = swz_word(fbase | (jh << 5));
    if constexpr (C == 3) {
      const float4 q0 = *reinterpret_cast<const float4*>(buf + a);
      const float4 q1 = *reinterpret_cast<const float4*>(buf + (a ^ 4));
      v[jh * 4 + 0] = make_float2(q0.x, q0.y); v[jh * 4 + 1] = make_float2(q0.z, q0.w);
      v[jh * 4 + 2] = make_float2(q1.x, q1.y); v[jh * 4 + 3] = make_float2(q1.z, q1.w);
    } else if constexpr (C == 2) {
      const float4 q0 = *reinterpret_cast<const float4*>(buf + a);
      v[jh * 2 + 0] = make_float2(q0.x, q0.y); v[jh * 2 + 1] = make_float2(q0.z, q0.w);
    } else if constexpr (C == 1) {
      v[jh] = *reinterpret_cast<const float2*>(buf + a);
    } else {
      if (jh & 1) v[jh >> 1].y = buf[a]; else v[jh >> 1].x = buf[a];
    }
  }
  if constexpr (C == 0) {
    // local bit 0 is index bit 5: that stage works inside each pair
#pragma unroll
    for (int e = 0; e < 32; ++e) v[e] = make_float2(v[e].x + v[e].y, v[e].x - v[e].y);
    stages2<0, 5>(v);
  } else {
    stages2<C - 1, 5>(v);      // pair-index bits [C-1, 5) are local bits [C, 6)
  }

  constexpr float norm = G::NORM;
  if (xr_out != nullptr) {       // stage export (uniform over the grid): x_r in fp32, nothing else
    if (live) {
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        float* dst = xr_out + token * K + findex(2 * e);
        if constexpr (C >= 1) {
          *reinterpret_cast<float2*>(dst) = make_float2(v[e].x * norm, v[e].y * norm);
        } else {
          dst[0] = v[e].x * norm;
          xr_out[token * K + findex(2 * e + 1)] = v[e].y * norm;
        }
      }
    }
    return;
  }

  // ---- per-token statistic (Eq. 5: max |x_r|; Eq. 6: mean |x_r|) ----
  float st;
  if constexpr (BITS == 8) {
    float m0 = 0.f, m1 = 0.f;
#pragma unroll
    for (int e = 0; e < 32; ++e) { m0 = fmaxf(m0, fabsf(v[e].x)); m1 = fmaxf(m1, fabsf(v[e].y)); }
    st = group_reduce<NT, true>(fmaxf(m0, m1), red_f, group, lane, warp_cta) * norm;
  } else {
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
      s0 += fabsf(v[e].x); s1 += fabsf(v[e].y); s2 += fabsf(v[e + 1].x); s3 += fabsf(v[e + 1].y);
    }
    const float s = group_reduce<NT, false>((s0 + s1) + (s2 + s3), red_f, group, lane, warp_cta);
    st = (s * norm) * (1.0f / (float)K);
  }
  constexpr float cq = (BITS == 8) ? 127.0f : kSqrt7;
  const float rq = __fdiv_rn(cq, st + eps) * norm;

  // ---- quantize; the low byte of (y + kMagic) is the code ----
  // (all reads of the exchange buffer happened before the barrier inside group_reduce)
  unsigned char* cbuf = reinterpret_cast<unsigned char*>(buf);
  const float2 rq2 = make_float2(rq, rq), magic2 = make_float2(kMagic, kMagic);
  uint32_t cb[32];               // per pair: code of .x in byte 0, code of .y in byte 1
#pragma unroll
  for (int e = 0; e < 32; ++e) {
    float2 y;
    if constexpr (BITS == 8) {
      y = __ffma2_rn(v[e], rq2, magic2);      // |x_r| * rq < 127: no clip needed
    } else {
      y = __fmul2_rn(v[e], rq2);
      y.x = fminf(fmaxf(y.x, -8.0f), 7.0f);
      y.y = fminf(fmaxf(y.y, -8.0f), 7.0f);
      y = __fadd2_rn(y, magic2);
    }
    cb[e] = __byte_perm(__float_as_uint(y.x), __float_as_uint(y.y), 0x0040);
  }
  if constexpr (C == 0) {
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      cbuf[swz_code(findex(2 * e))] = (unsigned char)(cb[e] & 0xFF);
      cbuf[swz_code(findex(2 * e + 1))] = (unsigned char)(cb[e] >> 8);
    }
  } else if constexpr (C == 1) {
#pragma unroll
    for (int e = 0; e < 32; ++e)
      *reinterpret_cast<unsigned short*>(cbuf + swz_code(findex(2 * e))) = (unsigned short)cb[e];
  } else if constexpr (C == 2) {
#pragma unroll
    for (int e = 0; e < 32; e += 2)
      *reinterpret_cast<uint32_t*>(cbuf + swz_code(findex(2 * e))) = __byte_perm(cb[e], cb[e + 1], 0x5410);
  } else {
#pragma unroll
    for (int e = 0; e < 32; e += 4)
      *reinterpret_cast<uint2*>(cbuf + swz_code(findex(2 * e))) =
          make_uint2(__byte_perm(cb[e], cb[e + 1], 0x5410), __byte_perm(cb[e + 2], cb[e + 3], 0x5410));
  }
  __syncthreads();

  // ---- coalesced copy-out: 4 chunks of 16 bytes per thread ----
  int csum = 0;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int q = tid + r * NT;
    const uint4 w = *reinterpret_cast<const uint4*>(cbuf + swz_code(q << 4));
    if (live) *reinterpret_cast<uint4*>(codes + token * K + ((size_t)q << 4)) = w;
    csum = __dp4a((int)w.x, 0x01010101, csum);
    csum = __dp4a((int)w.y, 0x01010101, csum);
    csum = __dp4a((int)w.z, 0x01010101, csum);
    csum = __dp4a((int)w.w, 0x01010101, csum);
  }
  if (codesum != nullptr) {      // uniform over the grid
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) csum += __shfl_xor_sync(0xffffffffu, csum, o);
    if (NT > 32) {
      if (lane == 0) red_i[warp_cta] = csum;
      __syncthreads();
      csum = 0;
#pragma unroll
      for (int w = 0; w < NT / 32; ++w) csum += red_i[group * (NT / 32) + w];
    }
    if (live && tid == 0) codesum[token] = csum;
  }
  if (live && tid == 0) scale[token] = __fdiv_rn(st, cq);
}

template <int M, int BITS>
int launch_one(const void* x, int T, float eps, int8_t* codes, float* scale, int32_t* codesum, float* xr_out,
               int32_t* zf, size_t zw, cudaStream_t s) {
  using G = Geometry<M>;
  const size_t smem = sizeof(float) * G::TPC * G::K;
  auto kern = fwht_quant_bf16_kernel<M, BITS>;
  if (smem > 48 * 1024) {
    static bool done = false;   // idempotent attribute; a race only repeats the call
    if (!done) {
      HBL_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      done = true;
    }
  }
  const int grid = (T + G::TPC - 1) / G::TPC;
  profile_before(KERNEL_ACT, s);
  kern<<<grid, G::THREADS, smem, s>>>(static_cast<const __nv_bfloat16*>(x), T, eps, codes, scale, codesum, xr_out,
                                      zf, zw);
  profile_after(KERNEL_ACT, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

}  // namespace

bool act_quant_bf16_supported(int K) { return K == 2048 || K == 4096 || K == 8192 || K == 16384; }

int launch_act_quant_bf16(const void* x, int T, int K, int bits, float eps, int8_t* codes, float* scale,
                          int32_t* codesum, float* xr_out, int32_t* zero_fill, size_t zero_fill_words,
                          cudaStream_t s) {
#define HBL_CASE(MM)                                                                                      \
  case (1 << MM):                                                                                         \
    return bits == 8 ? launch_one<MM, 8>(x, T, eps, codes, scale, codesum, xr_out, zero_fill, zero_fill_words, s) \
                     : launch_one<MM, 4>(x, T, eps, codes, scale, codesum, xr_out, zero_fill, zero_fill_words, s);
  switch (K) {
    HBL_CASE(11) HBL_CASE(12) HBL_CASE(13) HBL_CASE(14)
    default: return HBL_ERR_SHAPE;
  }
#undef HBL_CASE
}

}  // namespace hbl
