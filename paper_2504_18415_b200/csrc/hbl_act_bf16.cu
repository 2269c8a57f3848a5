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
//     transformed over index bits {0,2,3,4} -- including the two bits that live
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
#include "hbl_quant_rows.cuh"

namespace hbl {
namespace {

constexpr float kSqrt7 = 2.6457513110645906f;
constexpr float kMagic = 12582912.0f;          // 1.5 * 2^23: x + kMagic has rint(x) in its low mantissa bits

// ---- packed fp32 pairs, kept in 64-bit registers so that no pack/unpack moves are needed ----
typedef unsigned long long f32x2_t;

__device__ __forceinline__ f32x2_t pack2(float lo, float hi) {
  f32x2_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// (a, b) -> (a + b, a - b) on both halves.  The difference is fma(b, -1, a): one packed
// instruction with the same rounding as a subtraction.  `minus_one2` must live in a register
// pair for the whole kernel (see opaque_minus_one2): as a literal it is re-created before every use.
__device__ __forceinline__ void butterfly2(f32x2_t& a, f32x2_t& b, f32x2_t minus_one2) {
  f32x2_t s, d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(s) : "l"(a), "l"(b));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(b), "l"(minus_one2), "l"(a));
  a = s;
  b = d;
}
__device__ __forceinline__ f32x2_t opaque_minus_one2() {
  f32x2_t r;
  asm volatile("mov.b64 %0, 0xBF800000BF800000;" : "=l"(r));
  return r;
}
__device__ __forceinline__ f32x2_t fma2(f32x2_t a, f32x2_t b, f32x2_t c) {
  f32x2_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ f32x2_t mul2(f32x2_t a, f32x2_t b) {
  f32x2_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ float fma_sat(float a, float b, float c) {
  float r;
  asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// Butterfly stages over bits [B0, B1) of the pair index (v holds 32 pairs).
template <int B0, int B1>
__device__ __forceinline__ void stages2(f32x2_t (&v)[32], f32x2_t minus_one2) {
#pragma unroll
  for (int b = B0; b < B1; ++b) {
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      if ((e >> b) & 1) continue;
      butterfly2(v[e], v[e | (1 << b)], minus_one2);
    }
  }
}

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{0f00000000, 0f00000000, 0f00000000, 0f00000000};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Word address swizzle of a token's exchange buffer: toggles bit 2 with bits 5 and 8,
// which keeps every 4-word vector intact and makes the phase-0 vector stores and the
// final-phase loads of every supported M bank-conflict free.
__device__ __forceinline__ int swz_word(int a) { return a ^ ((((a >> 5) ^ (a >> 8)) & 1) << 2); }
// Byte address swizzle of the code staging area (keeps 16-byte chunks intact).
__device__ __forceinline__ int swz_code(int i) { return i ^ (((i >> 9) & 3) << 5); }

template <int M, int MIN_THREADS = 128>
struct Geometry {
  static constexpr int K = 1 << M;
  static constexpr int NT = K / 64;                       // threads per token
  static constexpr int THREADS = NT < MIN_THREADS ? MIN_THREADS : NT;
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

// What happens to the token before the transform sees it:
//   PRE_NONE  nothing;
//   PRE_NORM  RMS normalisation and a gain vector ("LN" of Eq. 7): x' = bf16(x * rsqrt(mean x^2 + norm_eps) * gain),
//             aux = gain [K], fp32 (PRE_NORM) or bf16 (PRE_NORM_BF16);
//   PRE_GLU   the SwishGLU product that feeds W_down: x' = bf16(SiLU(x) * aux), aux = the other projection's
//             output, bf16 [T, K] (x is the one that passes through SiLU).
enum { PRE_NONE = 0, PRE_NORM = 1, PRE_GLU = 2, PRE_NORM_BF16 = 3 };   // PRE_NORM_BF16: the same with a bf16 gain
// The body serves the tokens block * TPC ... of one input with a thread block of Geometry<M, MIN_THREADS>::THREADS
// threads: `smem` is TPC * K floats of shared memory aligned to 128 bytes (the swizzles toggle address
// bits up to 6), `red_f` / `red_i` are THREADS / 32 words each.
template <int M, int BITS, int PRE = PRE_NONE, int MIN_THREADS = 128>
__device__ __forceinline__ void fwht_quant_body(const __nv_bfloat16* __restrict__ x, int T, float eps, int8_t* __restrict__ codes,
                                                float* __restrict__ scale, int32_t* __restrict__ codesum,
                                                float* __restrict__ xr_out, const void* __restrict__ aux, float norm_eps,
                                                int packed, long block, float* smem, float* red_f, int* red_i) {
  using G = Geometry<M, MIN_THREADS>;
  constexpr int K = G::K, NT = G::NT, TPC = G::TPC, R = G::R, C = G::C, RUN = G::RUN;
  const int tid_cta = threadIdx.x;
  const int group = tid_cta / NT;
  const int tid = tid_cta % NT;
  const int lane = tid_cta & 31, warp_cta = tid_cta >> 5;
  const int warp = tid >> 5;                               // warp inside the token group
  const long token_raw = block * TPC + group;
  const bool live = token_raw < T;
  const long token = live ? token_raw : (long)T - 1;       // a dead group recomputes the last token, stores nothing
  float* buf = smem + (size_t)group * K;

  // ---- the 16x16 sign matrix as B fragments (two MMAs: output columns 0-7 and 8-15) ----
  // k-bit domain of the MMA: k0 = index bit 0, k1 k2 = index bits 3 4 (the lane's t), k3 = index bit 2.
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
  f32x2_t v[32];
  {
    const __nv_bfloat16* src = x + token * K + (warp << 8) + (lane << 3);
    uint4 raw[8];
#pragma unroll
    for (int c = 0; c < 8; ++c)
      raw[c] = __ldg(reinterpret_cast<const uint4*>(src + ((size_t)c << (M - 3))));
    if constexpr (PRE == PRE_GLU) {
      // SiLU(z) = z / (1 + exp(-z)) with the fast exponential and the fast division (relative error ~2^-21,
      // far inside the bf16 rounding that follows); exp(-z) overflows to +inf for very negative z and the
      // quotient becomes -0.
      const __nv_bfloat16* src2 = static_cast<const __nv_bfloat16*>(aux) + token * K + (warp << 8) + (lane << 3);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 up = __ldg(reinterpret_cast<const uint4*>(src2 + ((size_t)c << (M - 3))));
        const uint32_t u[4] = {up.x, up.y, up.z, up.w};
        uint32_t w[4] = {raw[c].x, raw[c].y, raw[c].z, raw[c].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float z0 = __uint_as_float(w[i] << 16), z1 = __uint_as_float(w[i] & 0xFFFF0000u);
          const float u0 = __uint_as_float(u[i] << 16), u1 = __uint_as_float(u[i] & 0xFFFF0000u);
          const float s0 = __fdividef(z0, 1.0f + __expf(-z0)), s1 = __fdividef(z1, 1.0f + __expf(-z1));
          const __nv_bfloat162 h = __floats2bfloat162_rn(s0 * u0, s1 * u1);
          w[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
        raw[c] = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
    if constexpr (PRE == PRE_NORM || PRE == PRE_NORM_BF16) {
      // mean square of the token in fp32 (64 values per thread, then the group), one reciprocal
      // square root, then (x * rstd) * gain rounded once to bf16 -- the transform's exact +-1
      // products need bf16 inputs, and bf16 is the type a model hands activations on in.
      // packed fp32 pairs throughout: a bf16 pair widens with one shift and one mask, and the squares,
      // the two multiplications and the rounding back to a bf16 pair are one instruction per pair each
      f32x2_t ss2 = pack2(0.f, 0.f);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint32_t w[4] = {raw[c].x, raw[c].y, raw[c].z, raw[c].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const f32x2_t v2 = pack2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
          ss2 = fma2(v2, v2, ss2);
        }
      }
      // (the widened values are not kept across the reduction: the compiler is made to widen again below)
#pragma unroll
      for (int c = 0; c < 8; ++c) asm volatile("" : "+r"(raw[c].x), "+r"(raw[c].y), "+r"(raw[c].z), "+r"(raw[c].w));
      float ss_lo, ss_hi;
      unpack2(ss2, ss_lo, ss_hi);
      const float ss = group_reduce<NT, false>(ss_lo + ss_hi, red_f, group, lane, warp_cta);
      const float rstd = __frcp_rn(__fsqrt_rn(__fmaf_rn(ss, 1.0f / (float)K, norm_eps)));
      const f32x2_t rstd2 = pack2(rstd, rstd);
      const size_t goff = (size_t)(warp << 8) + (lane << 3);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        f32x2_t g2[4];
        if constexpr (PRE == PRE_NORM_BF16) {                 // half the bytes to fetch from L2 per token
          const uint4 gb = __ldg(reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(aux) + goff + ((size_t)c << (M - 3))));
          const uint32_t gw[4] = {gb.x, gb.y, gb.z, gb.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) g2[i] = pack2(__uint_as_float(gw[i] << 16), __uint_as_float(gw[i] & 0xFFFF0000u));
        } else {
          const float* gp = static_cast<const float*>(aux) + goff + ((size_t)c << (M - 3));
          const float4 g0 = __ldg(reinterpret_cast<const float4*>(gp));
          const float4 g1 = __ldg(reinterpret_cast<const float4*>(gp + 4));
          g2[0] = pack2(g0.x, g0.y); g2[1] = pack2(g0.z, g0.w); g2[2] = pack2(g1.x, g1.y); g2[3] = pack2(g1.z, g1.w);
        }
        uint32_t w[4] = {raw[c].x, raw[c].y, raw[c].z, raw[c].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const f32x2_t v2 = pack2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
          float lo, hi;
          unpack2(mul2(mul2(v2, rstd2), g2[i]), lo, hi);      // (x * rstd) * gain, each product rounded to fp32
          const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
          w[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
        raw[c] = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      // A fragment, the loaded 16 bytes as they are: (x: m 0,1) rows g, k3 = 0; (y: m 2,3) rows g+8;
      // (z: m 4,5) k3 = 1; (w: m 6,7) both.  No register has to move between the load and the MMA, and each
      // MMA's four results are the two pairs that later leave in one 16-byte shared-memory store.
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        float d[4];
        mma_bf16_16816(d, raw[c].x, raw[c].y, raw[c].z, raw[c].w, hb[j][0], hb[j][1]);
        // d[2h + b] is position m = b + 2h + 4j; pair index p = h + 2j
        v[c * 4 + 2 * j] = pack2(d[0], d[1]);
        v[c * 4 + 2 * j + 1] = pack2(d[2], d[3]);
      }
    }
  }
  // pair index e = c*4 + p: bit 0 = index bit 1, bit 1 = index bit 2 (done by the MMA), bits 2..4 = the chunk bits
  const f32x2_t minus_one2 = opaque_minus_one2();
  stages2<0, 1>(v, minus_one2);
  stages2<2, 5>(v, minus_one2);

  // ---- exchange ----
  // Swizzled addresses are (thread part) ^ (compile-time part); the two parts meet in bit 2
  // only, so two base registers cover every case and the rest is an immediate offset.
  const uint32_t sbuf = static_cast<uint32_t>(__cvta_generic_to_shared(buf));
  {
    const uint32_t b0 = sbuf + 4u * swz_word((warp << 8) | (lane << 3));
    const uint32_t b1 = b0 ^ 16u;                          // word bit 2 toggled
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const int off = c << (M - 3);
      const bool flip = ((off >> 5) ^ (off >> 8)) & 1;     // the chunk's own swizzle contribution
      const uint32_t lo = (flip ? b1 : b0) + 4u * off, hi = (flip ? b0 : b1) + 4u * off;
      asm volatile("st.shared.v2.b64 [%0], {%1, %2};" ::"r"(lo), "l"(v[c * 4]), "l"(v[c * 4 + 1]) : "memory");
      asm volatile("st.shared.v2.b64 [%0], {%1, %2};" ::"r"(hi), "l"(v[c * 4 + 2]), "l"(v[c * 4 + 3]) : "memory");
    }
  }
  __syncthreads();

  // ---- final layout: local j (6 bits): low C bits = index bits [0,C), high R bits = index bits [5,5+R) ----
  const int fbase = ((tid & ((1 << (5 - C)) - 1)) << C) | ((tid >> (5 - C)) << (M - 3));
  auto findex = [&](int j) { return fbase | (j & (RUN - 1)) | ((j >> C) << 5); };
  {
    const uint32_t f0 = sbuf + 4u * swz_word(fbase);
    const uint32_t f1 = f0 ^ 16u;
#pragma unroll
    for (int jh = 0; jh < (1 << R); ++jh) {
      const int off = jh << 5;
      const bool flip = ((off >> 5) ^ (off >> 8)) & 1;
      const uint32_t a = (flip ? f1 : f0) + 4u * off, a_hi = (flip ? f0 : f1) + 4u * off;
      if constexpr (C == 3) {
        asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(v[jh * 4]), "=l"(v[jh * 4 + 1]) : "r"(a));
        asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(v[jh * 4 + 2]), "=l"(v[jh * 4 + 3]) : "r"(a_hi));
      } else if constexpr (C == 2) {
        asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(v[jh * 2]), "=l"(v[jh * 2 + 1]) : "r"(a));
      } else if constexpr (C == 1) {
        asm volatile("ld.shared.b64 %0, [%1];" : "=l"(v[jh]) : "r"(a));
      } else {
        if ((jh & 1) == 0) {                               // local bit 0 = index bit 5: elements jh, jh+1 form a pair
          const int off1 = (jh + 1) << 5;
          const bool flip1 = ((off1 >> 5) ^ (off1 >> 8)) & 1;
          float lo, hi;
          asm volatile("ld.shared.f32 %0, [%1];" : "=f"(lo) : "r"(a));
          asm volatile("ld.shared.f32 %0, [%1];" : "=f"(hi) : "r"((flip1 ? f1 : f0) + 4u * off1));
          v[jh >> 1] = pack2(lo, hi);
        }
      }
    }
  }
  // All stages but the last one (pair-index bit 4).
  if constexpr (C == 0) {
    // local bit 0 is index bit 5: that stage works inside each pair
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      float lo, hi;
      unpack2(v[e], lo, hi);
      v[e] = pack2(lo + hi, lo - hi);
    }
    stages2<0, 4>(v, minus_one2);
  } else {
    stages2<C - 1, 4>(v, minus_one2);      // pair-index bits [C-1, 5) are local bits [C, 6)
  }
  // Last stage, with the statistic's raw material taken from its inputs:
  //   |a+b| + |a-b| = 2 max(|a|,|b|)   and   max(|a+b|,|a-b|) = |a| + |b|.
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int e = 0; e < 16; ++e) {
    float ax, ay, bx, by;
    unpack2(v[e], ax, ay);
    unpack2(v[e + 16], bx, by);
    if constexpr (BITS == 8) {
      s0 = fmaxf(s0, fabsf(ax) + fabsf(bx));
      s1 = fmaxf(s1, fabsf(ay) + fabsf(by));
    } else {
      s0 += fmaxf(fabsf(ax), fabsf(bx));
      s1 += fmaxf(fabsf(ay), fabsf(by));
    }
    butterfly2(v[e], v[e + 16], minus_one2);
  }

  constexpr float norm = G::NORM;
  if constexpr (BITS == 0) {
    // Transform only, bf16 out (the backward pass of the transform, Eq. 8, is this same product applied
    // to the gradient): `codes` is the bf16 output [T, K].  One rounding, fp32 -> bf16, after the scale.
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(codes) + token * K;
    if (live) {
      if constexpr (C == 0) {
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          float lo, hi;
          unpack2(v[e], lo, hi);
          out[findex(2 * e)] = __float2bfloat16_rn(lo * norm);
          out[findex(2 * e + 1)] = __float2bfloat16_rn(hi * norm);
        }
      } else {
        constexpr int PAIRS = RUN / 2;                       // pairs per run of consecutive elements
#pragma unroll
        for (int r = 0; r < 32 / PAIRS; ++r) {
          uint32_t w[PAIRS];
#pragma unroll
          for (int q = 0; q < PAIRS; ++q) {
            float lo, hi;
            unpack2(v[r * PAIRS + q], lo, hi);
            const __nv_bfloat162 h = __floats2bfloat162_rn(lo * norm, hi * norm);
            w[q] = *reinterpret_cast<const uint32_t*>(&h);
          }
          __nv_bfloat16* dst = out + findex(r * RUN);
          if constexpr (PAIRS == 4) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
          else if constexpr (PAIRS == 2) *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
          else *reinterpret_cast<uint32_t*>(dst) = w[0];
        }
      }
    }
    return;
  }
  if (xr_out != nullptr) {       // stage export (uniform over the grid): x_r in fp32, nothing else
    if (live) {
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        float lo, hi;
        unpack2(v[e], lo, hi);
        float* dst = xr_out + token * K + findex(2 * e);
        if constexpr (C >= 1) {
          *reinterpret_cast<float2*>(dst) = make_float2(lo * norm, hi * norm);
        } else {
          dst[0] = lo * norm;
          xr_out[token * K + findex(2 * e + 1)] = hi * norm;
        }
      }
    }
    return;
  }

  // ---- per-token statistic (Eq. 5: max |x_r|; Eq. 6: mean |x_r|) ----
  float st;
  if constexpr (BITS == 8) {
    st = group_reduce<NT, true>(fmaxf(s0, s1), red_f, group, lane, warp_cta) * norm;
  } else {
    const float s = group_reduce<NT, false>(s0 + s1, red_f, group, lane, warp_cta);
    st = ((2.0f * s) * norm) * (1.0f / (float)K);
  }
  constexpr float cq = (BITS == 8) ? 127.0f : kSqrt7;
  const float rq = __fdiv_rn(cq, st + eps) * norm;

  // ---- quantize; the low byte of (y + kMagic) is the code ----
  // (all reads of the exchange buffer happened before the barrier inside group_reduce)
  unsigned char* cbuf = reinterpret_cast<unsigned char*>(buf);
  uint32_t cb[32];               // per pair: code of the low element in byte 0, of the high one in byte 1
  if constexpr (BITS == 8) {
    const f32x2_t rq2 = pack2(rq, rq), magic2 = pack2(kMagic, kMagic);
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      float lo, hi;
      unpack2(fma2(v[e], rq2, magic2), lo, hi);   // |x_r| * rq < 127.5: no clip needed
      cb[e] = __byte_perm(__float_as_uint(lo), __float_as_uint(hi), 0x0040);
    }
  } else {
    // RoundClip(y, -8, 7) with y = x_r * rq: u = sat(y/15 + 8/15) is the clip (to [0,1]),
    // 15 u - 8 + kMagic the rounding.  The two extra roundings move y by < 2e-6.
    const float rq15 = rq * (1.0f / 15.0f);
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      float lo, hi;
      unpack2(v[e], lo, hi);
      lo = __fmaf_rn(fma_sat(lo, rq15, 8.0f / 15.0f), 15.0f, kMagic - 8.0f);
      hi = __fmaf_rn(fma_sat(hi, rq15, 8.0f / 15.0f), 15.0f, kMagic - 8.0f);
      cb[e] = __byte_perm(__float_as_uint(lo), __float_as_uint(hi), 0x0040);
    }
  }
  // Staging byte address of element fbase | off(j): swz_code adds (index bits 9,10) << 5 onto bits 5,6,
  // which always belong to off(j).  The thread's share of that is a 2-bit value tt, so four base
  // registers (one per value of the offset's own bits 5,6) leave only immediates per store.
  uint32_t cbase[4];
  {
    const uint32_t tt = (uint32_t)(fbase >> 9) & 3u;
#pragma unroll
    for (int p = 0; p < 4; ++p) cbase[p] = sbuf + (uint32_t)fbase + (((uint32_t)p ^ tt) << 5);
  }
  auto caddr = [&](int j) {
    const int off = (j & (RUN - 1)) | ((j >> C) << 5);
    const int x = off ^ (((off >> 9) & 3) << 5);
    return cbase[(x >> 5) & 3] + (uint32_t)(x & ~96);
  };
  if constexpr (C == 0) {
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      asm volatile("st.shared.u8 [%0], %1;" ::"r"(caddr(2 * e)), "r"(cb[e]) : "memory");
      asm volatile("st.shared.u8 [%0], %1;" ::"r"(caddr(2 * e + 1)), "r"(cb[e] >> 8) : "memory");
    }
  } else if constexpr (C == 1) {
#pragma unroll
    for (int e = 0; e < 32; ++e) asm volatile("st.shared.u16 [%0], %1;" ::"r"(caddr(2 * e)), "h"((unsigned short)cb[e]) : "memory");
  } else if constexpr (C == 2) {
#pragma unroll
    for (int e = 0; e < 32; e += 2)
      asm volatile("st.shared.u32 [%0], %1;" ::"r"(caddr(2 * e)), "r"(__byte_perm(cb[e], cb[e + 1], 0x5410)) : "memory");
  } else {
#pragma unroll
    for (int e = 0; e < 32; e += 4)
      asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(caddr(2 * e)), "r"(__byte_perm(cb[e], cb[e + 1], 0x5410)),
                   "r"(__byte_perm(cb[e + 2], cb[e + 3], 0x5410)) : "memory");
  }
  __syncthreads();

  if (BITS == 4 && packed) {     // uniform over the grid
    // ---- INT4 codes two per byte: 2 chunks of 16 bytes (32 codes each) per thread.  The 32-bit word g of a
    //      token's row covers elements 8g .. 8g+7: byte b = (q[8g+b] + 8) | (q[8g+b+4] + 8) << 4 ----
    auto pack8 = [](uint32_t first4, uint32_t next4) {
      return ((first4 & 0x0F0F0F0Fu) | ((next4 & 0x0F0F0F0Fu) << 4)) ^ 0x88888888u;   // q & 15 -> (q + 8) & 15
    };
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int pc = tid + r * NT;
      const uint4 a = *reinterpret_cast<const uint4*>(cbuf + swz_code((2 * pc) << 4));
      const uint4 b = *reinterpret_cast<const uint4*>(cbuf + swz_code((2 * pc + 1) << 4));
      const uint4 o = make_uint4(pack8(a.x, a.y), pack8(a.z, a.w), pack8(b.x, b.y), pack8(b.z, b.w));
      if (live) *reinterpret_cast<uint4*>(codes + token * (K / 2) + ((size_t)pc << 4)) = o;
    }
    if (live && tid == 0) scale[token] = __fdiv_rn(st, cq);
    return;
  }
  // ---- coalesced copy-out: 4 chunks of 16 bytes per thread ----
  int csum = 0;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int q = tid + r * NT;
    const uint4 w = *reinterpret_cast<const uint4*>(cbuf + swz_code(q << 4));
    if (live) *reinterpret_cast<uint4*>(codes + token * K + ((size_t)q << 4)) = w;
    if (codesum != nullptr) {
      csum = __dp4a((int)w.x, 0x01010101, csum);
      csum = __dp4a((int)w.y, 0x01010101, csum);
      csum = __dp4a((int)w.z, 0x01010101, csum);
      csum = __dp4a((int)w.w, 0x01010101, csum);
    }
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

template <int M, int BITS, int PRE = PRE_NONE>
__global__ void __launch_bounds__(Geometry<M>::THREADS, 768 / Geometry<M>::THREADS)
fwht_quant_bf16_kernel(const __nv_bfloat16* __restrict__ x, int T, float eps, int8_t* __restrict__ codes,
                       float* __restrict__ scale, int32_t* __restrict__ codesum, float* __restrict__ xr_out,
                       int32_t* __restrict__ zero_fill, size_t zero_words, const void* __restrict__ aux,
                       float norm_eps, int packed) {
  constexpr int THREADS = Geometry<M>::THREADS;
  extern __shared__ __align__(128) float smem[];
  __shared__ float red_f[THREADS / 32];
  __shared__ int red_i[THREADS / 32];
  // A kernel launched as a programmatic dependent of this one may start now; it waits (griddepcontrol.wait)
  // before it touches anything written here.
  grid_launch_dependents();
  if (zero_fill != nullptr) {   // side job: clear the caller's scratch words
    for (size_t i = (size_t)blockIdx.x * THREADS + threadIdx.x; i < zero_words; i += (size_t)gridDim.x * THREADS)
      zero_fill[i] = 0;
  }
  fwht_quant_body<M, BITS, PRE>(x, T, eps, codes, scale, codesum, xr_out, aux, norm_eps, packed, (long)blockIdx.x, smem,
                                red_f, red_i);
  grid_dependency_wait();   // chain: this kernel is complete only when the one before it is
}

template <int M, int BITS, int PRE = PRE_NONE>
int launch_one(const void* x, int T, float eps, int8_t* codes, float* scale, int32_t* codesum, float* xr_out,
               int32_t* zf, size_t zw, cudaStream_t s, const void* aux = nullptr, float norm_eps = 0.f, bool packed = false) {
  using G = Geometry<M>;
  const size_t smem = sizeof(float) * G::TPC * G::K;
  auto kern = fwht_quant_bf16_kernel<M, BITS, PRE>;
  if (smem > 48 * 1024) HBL_ALLOW_DYNAMIC_SMEM(kern, smem);
  const int grid = (T + G::TPC - 1) / G::TPC;
  profile_before(KERNEL_ACT, s);
  HBL_CUDA_OK(launch_dependent(kern, dim3(grid), dim3(G::THREADS), smem, s, static_cast<const __nv_bfloat16*>(x), T, eps,
                               codes, scale, codesum, xr_out, zf, zw, aux, norm_eps, (int)packed));
  profile_after(KERNEL_ACT, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

}  // namespace

int launch_norm_act_quant_bf16(const void* x, const void* gain, int gain_dtype, float norm_eps, int T, int K, int bits,
                               float eps, int8_t* codes, float* scale, int32_t* codesum, float* xr_out,
                               int32_t* zero_fill, size_t zero_fill_words, cudaStream_t s, bool packed) {
#define HBL_CASE(MM)                                                                                              \
  case (1 << MM):                                                                                                 \
    if (gain_dtype == HBL_BF16)                                                                                   \
      return bits == 8 ? launch_one<MM, 8, PRE_NORM_BF16>(x, T, eps, codes, scale, codesum, xr_out, zero_fill, zero_fill_words, s, gain, norm_eps, packed) \
                       : launch_one<MM, 4, PRE_NORM_BF16>(x, T, eps, codes, scale, codesum, xr_out, zero_fill, zero_fill_words, s, gain, norm_eps, packed); \
    return bits == 8 ? launch_one<MM, 8, PRE_NORM>(x, T, eps, codes, scale, codesum, xr_out, zero_fill, zero_fill_words, s, gain, norm_eps, packed) \
                     : launch_one<MM, 4, PRE_NORM>(x, T, eps, codes, scale, codesum, xr_out, zero_fill, zero_fill_words, s, gain, norm_eps, packed);
  switch (K) {
    HBL_CASE(11) HBL_CASE(12) HBL_CASE(13) HBL_CASE(14)
    default: return HBL_ERR_SHAPE;
  }
#undef HBL_CASE
}

int launch_glu_act_quant_bf16(const void* gate, const void* up, int T, int K, int bits, float eps, int8_t* codes,
                              float* scale, int32_t* codesum, float* xr_out, int32_t* zero_fill, size_t zero_fill_words,
                              cudaStream_t s, bool packed) {
#define HBL_CASE(MM)                                                                                              \
  case (1 << MM):                                                                                                 \
    return bits == 8 ? launch_one<MM, 8, PRE_GLU>(gate, T, eps, codes, scale, codesum, xr_out, zero_fill, zero_fill_words, s, up, 0.f, packed) \
                     : launch_one<MM, 4, PRE_GLU>(gate, T, eps, codes, scale, codesum, xr_out, zero_fill, zero_fill_words, s, up, 0.f, packed);
  switch (K) {
    HBL_CASE(11) HBL_CASE(12) HBL_CASE(13) HBL_CASE(14)
    default: return HBL_ERR_SHAPE;
  }
#undef HBL_CASE
}

int launch_hadamard_bf16(const void* x, int T, int K, void* out, cudaStream_t s) {
  if (T <= 0) return HBL_OK;
  int8_t* o = static_cast<int8_t*>(out);
  switch (K) {
    case 2048: return launch_one<11, 0>(x, T, 1.0f, o, nullptr, nullptr, nullptr, nullptr, 0, s);
    case 4096: return launch_one<12, 0>(x, T, 1.0f, o, nullptr, nullptr, nullptr, nullptr, 0, s);
    case 8192: return launch_one<13, 0>(x, T, 1.0f, o, nullptr, nullptr, nullptr, nullptr, 0, s);
    case 16384: return launch_one<14, 0>(x, T, 1.0f, o, nullptr, nullptr, nullptr, nullptr, 0, s);
    default: return HBL_ERR_SHAPE;
  }
}

bool act_quant_bf16_supported(int K) { return K == 2048 || K == 4096 || K == 8192 || K == 16384; }

int launch_act_quant_bf16(const void* x, int T, int K, int bits, float eps, int8_t* codes, float* scale,
                          int32_t* codesum, float* xr_out, int32_t* zero_fill, size_t zero_fill_words,
                          cudaStream_t s, bool packed) {
#define HBL_CASE(MM)                                                                                      \
  case (1 << MM):                                                                                         \
    return bits == 8 ? launch_one<MM, 8>(x, T, eps, codes, scale, codesum, xr_out, zero_fill, zero_fill_words, s, nullptr, 0.f, packed) \
                     : launch_one<MM, 4>(x, T, eps, codes, scale, codesum, xr_out, zero_fill, zero_fill_words, s, nullptr, 0.f, packed);
  switch (K) {
    HBL_CASE(11) HBL_CASE(12) HBL_CASE(13) HBL_CASE(14)
    default: return HBL_ERR_SHAPE;
  }
#undef HBL_CASE
}

// ---- several bf16 inputs of the same token count in one launch ----
// A decoder block quantizes four inputs before its contraction.  As four kernels they are four dependent
// launches, each a microsecond or two of latency that a handful of tokens cannot hide; here every input gets a
// range of thread blocks of one grid.  Inputs with the transform run fwht_quant_body (K = 2^11..2^14), inputs
// without it quant_rows_bf16_body (K a multiple of 128, at most 16384), all with 256 threads per block.
namespace {

constexpr int kMultiThreads = 256;
constexpr size_t kMultiMaxSmem = sizeof(float) * 16384;

struct ActMultiParams {
  ActJob job[kMaxActJobs];
  int first_block[kMaxActJobs + 1];   // input j owns blocks [first_block[j], first_block[j + 1])
  int nt[kMaxActJobs];                // threads per token of an input without the transform
  int n, T;
  float eps;
  int32_t* zero_fill;
  size_t zero_words;
  unsigned* ready;                    // per input: thread blocks that have written their codes (nullptr: not counted)
};

// Last thing a thread block does: its stores are made visible, then one thread counts the block in.
__device__ __forceinline__ void count_block_in(unsigned* counter) {
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) atomicAdd(counter, 1u);
}

template <int BITS>
__global__ void __launch_bounds__(kMultiThreads, 3)
act_multi_bf16_kernel(const __grid_constant__ ActMultiParams p) {
  extern __shared__ __align__(128) float smem[];
  __shared__ float red_f[16];
  __shared__ int red_i[16];
  grid_launch_dependents();   // the contraction that follows may start and fetch its first weights
  if (p.zero_fill != nullptr)
    for (size_t i = (size_t)blockIdx.x * kMultiThreads + threadIdx.x; i < p.zero_words; i += (size_t)gridDim.x * kMultiThreads)
      p.zero_fill[i] = 0;
  int j = 0;
  while (j + 1 < p.n && (int)blockIdx.x >= p.first_block[j + 1]) ++j;
  const ActJob& job = p.job[j];
  const long block = (long)blockIdx.x - p.first_block[j];
  const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(job.x);
  if (!job.use_hadamard) {
    quant_rows_bf16_body<BITS>(x, p.T, job.K, p.nt[j], p.eps, job.codes, job.scale, job.codesum, 0, block, red_f, red_i);
    if (p.ready != nullptr) count_block_in(p.ready + j);
    grid_dependency_wait();   // chain: this kernel is complete only when the one before it is
    return;
  }
#define HBL_CASE(MM)                                                                                                \
  case (1 << MM):                                                                                                   \
    fwht_quant_body<MM, BITS, PRE_NONE, kMultiThreads>(x, p.T, p.eps, job.codes, job.scale, job.codesum, nullptr, nullptr, \
                                                       0.f, 0, block, smem, red_f, red_i);                          \
    break;
  switch (job.K) {
    HBL_CASE(11) HBL_CASE(12) HBL_CASE(13) HBL_CASE(14)
    default: break;
  }
#undef HBL_CASE
  if (p.ready != nullptr) count_block_in(p.ready + j);
  grid_dependency_wait();
}

}  // namespace

bool act_multi_bf16_supported(const ActJob* jobs, int n_jobs) {
  if (n_jobs < 1 || n_jobs > kMaxActJobs) return false;
  for (int j = 0; j < n_jobs; ++j) {
    const int K = jobs[j].K;
    if (jobs[j].use_hadamard ? !act_quant_bf16_supported(K) : (K % 128 != 0 || K > 16384)) return false;
  }
  return true;
}

int launch_act_multi_bf16(const ActJob* jobs, int n_jobs, int T, int bits, float eps, int32_t* zero_fill,
                          size_t zero_fill_words, cudaStream_t s, unsigned* ready, unsigned* blocks_out) {
  if (T <= 0) return HBL_OK;
  if (!act_multi_bf16_supported(jobs, n_jobs)) return HBL_ERR_SHAPE;
  if (bits != 4 && bits != 8) return HBL_ERR_BITS;
  ActMultiParams p{};
  size_t smem = 0;
  int blocks = 0;
  for (int j = 0; j < n_jobs; ++j) {
    p.job[j] = jobs[j];
    p.first_block[j] = blocks;
    const int K = jobs[j].K;
    int tpc;
    if (jobs[j].use_hadamard) {
      const int nt = K / 64;
      tpc = nt < kMultiThreads ? kMultiThreads / nt : 1;
      const size_t need = sizeof(float) * (size_t)tpc * K;
      if (need > smem) smem = need;
    } else {
      p.nt[j] = ((K / 8 + 7) / 8 + 31) / 32 * 32;           // eight 16-byte chunks per thread, whole warps
      tpc = kMultiThreads / p.nt[j];
    }
    blocks += (T + tpc - 1) / tpc;
    if (blocks_out != nullptr) blocks_out[j] = (unsigned)((T + tpc - 1) / tpc);
  }
  p.first_block[n_jobs] = blocks;
  p.n = n_jobs;
  p.T = T;
  p.eps = eps;
  p.zero_fill = zero_fill;
  p.zero_words = zero_fill_words;
  p.ready = ready;
  auto kern = bits == 8 ? act_multi_bf16_kernel<8> : act_multi_bf16_kernel<4>;
  // (the attribute is set once per device, to the most any supported input needs: 2^14 floats)
  if (bits == 8) HBL_ALLOW_DYNAMIC_SMEM(act_multi_bf16_kernel<8>, kMultiMaxSmem);
  else HBL_ALLOW_DYNAMIC_SMEM(act_multi_bf16_kernel<4>, kMultiMaxSmem);
  profile_before(KERNEL_ACT, s);
  HBL_CUDA_OK(launch_dependent(kern, dim3(blocks), dim3(kMultiThreads), smem, s, p));
  profile_after(KERNEL_ACT, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

}  // namespace hbl
