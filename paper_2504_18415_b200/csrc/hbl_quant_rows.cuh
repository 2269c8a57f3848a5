// bf16 input, no transform (Eq. 5-6 on x itself), any K that is a multiple of 128: bound by HBM, so the code
// spends as few instructions per element as it can.  A group of NT threads (a multiple of 32) owns a token;
// thread t holds the 16-byte chunks t, t + NT, ... (up to eight: 64 elements in registers), so every load and
// every 8-byte store of codes is coalesced and the token is read once.  Rounding is the magic-number add
// (x * rq + 1.5 * 2^23 has rint(x * rq) in its low mantissa bits: no float-to-int conversion, which runs at a
// quarter of the rate); the INT8 maximum is taken on bf16 pairs (exact); the sum of codes is a byte dot product.
//
// The body is a device function: a thread block of blockDim.x threads serves
// blockDim.x / NT tokens starting at token block * (blockDim.x / NT); `red_f` and `red_i` are 16 words of shared
// memory each.  Used by the single-input kernel and by the kernel that serves several inputs in one launch.
#pragma once
#include "hbl_common.cuh"

namespace hbl {

constexpr float kRowsSqrt7 = 2.6457513110645906f;
constexpr float kRowsMagic = 12582912.0f;          // 1.5 * 2^23: y + kRowsMagic has rint(y) in its low mantissa bits
__device__ __forceinline__ float rows_bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float rows_bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ float fma_sat_f32(float a, float b, float c) {
  float r;
  asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

template <int BITS>
__device__ __forceinline__ void quant_rows_bf16_body(const __nv_bfloat16* __restrict__ x, int T, int K, int NT, float eps,
                                                     int8_t* __restrict__ codes, float* __restrict__ scale,
                                                     int32_t* __restrict__ codesum, int packed, long block,
                                                     float* red_f, int* red_i) {
  const int tid_cta = threadIdx.x, lane = tid_cta & 31, warp = tid_cta >> 5;
  const int TPC = blockDim.x / NT, W = NT >> 5;                     // token groups per CTA, warps per group
  const int group = tid_cta / NT, tid = tid_cta - group * NT;
  const int warp0 = group * W;
  const long token_raw = block * TPC + group;
  const bool live = token_raw < T;
  const long token = live ? token_raw : (long)T - 1;                // a dead group redoes the last token, stores nothing
  const int n_chunks = K >> 3;

  uint4 raw[8];
  {
    const uint4* src = reinterpret_cast<const uint4*>(x + token * K);
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const int chunk = c * NT + tid;
      raw[c] = chunk < n_chunks ? __ldg(src + chunk) : make_uint4(0u, 0u, 0u, 0u);
    }
  }

  // ---- per-token statistic (Eq. 5: max |x|; Eq. 6: mean |x|) ----
  float st;
  if constexpr (BITS == 8) {
    uint32_t m2 = 0;                                                // a pair of bf16 maxima of |x|
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const uint32_t w[4] = {raw[c].x, raw[c].y, raw[c].z, raw[c].w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t a = w[i] & 0x7FFF7FFFu;
        const __nv_bfloat162 h = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&m2), *reinterpret_cast<const __nv_bfloat162*>(&a));
        m2 = *reinterpret_cast<const uint32_t*>(&h);
      }
    }
    st = fmaxf(rows_bf16_lo(m2), rows_bf16_hi(m2));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) st = fmaxf(st, __shfl_xor_sync(0xffffffffu, st, o));
  } else {
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const uint32_t w[4] = {raw[c].x, raw[c].y, raw[c].z, raw[c].w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        s0 += fabsf(rows_bf16_lo(w[i]));
        s1 += fabsf(rows_bf16_hi(w[i]));
      }
    }
    st = s0 + s1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) st += __shfl_xor_sync(0xffffffffu, st, o);
  }
  if constexpr (BITS != 8) {
    // the widened values are not worth keeping across the reduction (64 registers): make the compiler
    // widen again below
#pragma unroll
    for (int c = 0; c < 8; ++c) asm volatile("" : "+r"(raw[c].x), "+r"(raw[c].y), "+r"(raw[c].z), "+r"(raw[c].w));
  }
  if (lane == 0) red_f[warp] = st;
  __syncthreads();
  st = red_f[warp0];
  for (int w = 1; w < W; ++w) st = (BITS == 8) ? fmaxf(st, red_f[warp0 + w]) : st + red_f[warp0 + w];
  if constexpr (BITS != 8) st = __fdiv_rn(st, (float)K);
  constexpr float cq = (BITS == 8) ? 127.0f : kRowsSqrt7;
  const float rq = __fdiv_rn(cq, st + eps);

  // ---- quantize: eight codes per chunk, one 8-byte store ----
  int csum = 0;
  int8_t* dst = codes + token * K;
  const float rq15 = rq * (1.0f / 15.0f);
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const uint32_t w[4] = {raw[c].x, raw[c].y, raw[c].z, raw[c].w};
    uint32_t h[4];                                                  // two codes each, in bytes 0 and 1
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float lo = rows_bf16_lo(w[i]), hi = rows_bf16_hi(w[i]);
      if constexpr (BITS == 8) {                                    // |x| rq < 127.5: nothing to clip
        lo = __fmaf_rn(lo, rq, kRowsMagic);
        hi = __fmaf_rn(hi, rq, kRowsMagic);
      } else {
        // RoundClip(y, -8, 7) with y = x rq: u = sat(y / 15 + 8 / 15) is the clip (to [0, 1]), 15 u - 8 + magic
        // the rounding; the two extra roundings move y by < 2e-6
        lo = __fmaf_rn(fma_sat_f32(lo, rq15, 8.0f / 15.0f), 15.0f, kRowsMagic - 8.0f);
        hi = __fmaf_rn(fma_sat_f32(hi, rq15, 8.0f / 15.0f), 15.0f, kRowsMagic - 8.0f);
      }
      h[i] = __byte_perm(__float_as_uint(lo), __float_as_uint(hi), 0x0040);
    }
    const uint32_t q0 = __byte_perm(h[0], h[1], 0x5410), q1 = __byte_perm(h[2], h[3], 0x5410);
    const int chunk = c * NT + tid;
    if (chunk < n_chunks) {
      csum = __dp4a((int)q0, 0x01010101, csum);
      csum = __dp4a((int)q1, 0x01010101, csum);
      if (BITS == 4 && packed) {
        // INT4 codes two per byte: this chunk is the 32-bit word `chunk` of the token's K / 2 bytes,
        // byte b = (q[b] + 8) | (q[b + 4] + 8) << 4
        const uint32_t pk = ((q0 & 0x0F0F0F0Fu) | ((q1 & 0x0F0F0F0Fu) << 4)) ^ 0x88888888u;
        if (live) *reinterpret_cast<uint32_t*>(codes + token * (K / 2) + (size_t)chunk * 4) = pk;
      } else if (live) {
        *reinterpret_cast<uint2*>(dst + (size_t)chunk * 8) = make_uint2(q0, q1);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) csum += __shfl_xor_sync(0xffffffffu, csum, o);
  if (lane == 0) red_i[warp] = csum;
  __syncthreads();
  if (live && tid == 0) {
    int t = 0;
    for (int w = 0; w < W; ++w) t += red_i[warp0 + w];
    scale[token] = __fdiv_rn(st, cq);
    if (codesum != nullptr) codesum[token] = t;
  }
}

}  // namespace hbl
