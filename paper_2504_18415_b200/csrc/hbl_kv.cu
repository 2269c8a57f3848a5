// Low-bit attention states (BitNet v2, section 3.1, Tables 2-3): the Q, K and V heads are quantized after the
// rotary embedding to unsigned integers with the absmax function, 4-bit or 3-bit for the KV cache, and the K/V
// heads of the [BOS] token stay at 8 bits.  The paper prints no formula for it; this is Eq. 5's absmax quantizer
// at b bits, one statistic per head of each token, stored with an offset so that the code is unsigned:
//
//   gamma = max_d |x[d]|,  q = RoundClip((2^(b-1) - 1) / (gamma + eps) * x, -2^(b-1), 2^(b-1) - 1),
//   u = q + 2^(b-1),       s = gamma / (2^(b-1) - 1)          (x ~ s * (u - 2^(b-1)))
//
// Bound by HBM: 2 bytes read and b/8 bytes written per element.  A thread takes 8 consecutive elements of one
// head (one 16-byte load), the head_dim / 8 lanes of a head share the maximum by shuffles, and the codes of a
// head leave as one contiguous run of head_dim * b / 8 bytes.
#include "hbl_common.cuh"

namespace hbl {
namespace {

constexpr int kThreads = 256;

constexpr int kUnroll = 4;                                   // 16-byte chunks in flight per thread
constexpr float kMagic = 12582912.0f;                        // 1.5 * 2^23: x + kMagic has rint(x) in its low mantissa bits

// Codes of 8 consecutive elements for width BITS, as the low bytes of u[0..7], from the fp32 values f and the
// head's factor rq = c / (gamma + eps), c = 2^(BITS-1) - 1: IEEE fp32 product, round to nearest even.  No clip
// is needed: |x| <= gamma gives |v| <= c gamma / (gamma + eps) < c, so the rounded value already lies inside
// [-2^(BITS-1), 2^(BITS-1) - 1].  The rounding is the magic-number add (|v| is far below 2^22), with the offset
// 2^(BITS-1) folded into the constant: the low byte of the sum is the unsigned code.
template <int BITS>
__device__ __forceinline__ void codes8(const float (&f)[8], float rq, uint32_t (&u)[8]) {
  constexpr int HALF = 1 << (BITS - 1);
#pragma unroll
  for (int i = 0; i < 8; ++i) u[i] = __float_as_uint(__fadd_rn(__fmul_rn(rq, f[i]), kMagic + (float)HALF));
}
// The low bytes of four words as one word (byte i = low byte of u[i]).
__device__ __forceinline__ uint32_t low_bytes(uint32_t u0, uint32_t u1, uint32_t u2, uint32_t u3) {
  return __byte_perm(__byte_perm(u0, u1, 0x0040), __byte_perm(u2, u3, 0x0040), 0x5410);
}
__device__ __forceinline__ void widen8(const uint4& raw, float (&f)[8]) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}

// LPH = lanes per head = head_dim / 8.  A thread block takes tiles of kUnroll x kThreads chunks; a thread's
// kUnroll loads are issued before any arithmetic.  The two IEEE divisions of a head (c / (gamma + eps) and
// gamma / c) are what costs most instructions here, and a warp pays for a division whatever the number of its
// lanes that need it: so the maxima of all heads a warp holds in a tile (kUnroll x 32 / LPH of them) are
// gathered one per lane, divided once, and the factors handed back by shuffles.
template <int BITS, int LPH>
__global__ void __launch_bounds__(kThreads)
kv_quant_kernel(const uint4* __restrict__ x, long n_rows, int n_heads, int seq_len, float eps,
                unsigned char* __restrict__ codes, float* __restrict__ scale, unsigned char* __restrict__ bos_codes,
                float* __restrict__ bos_scale) {
  constexpr int HALF = 1 << (BITS - 1);
  constexpr int ROW_BYTES = LPH * BITS;                     // head_dim * BITS / 8
  constexpr long TILE = (long)kUnroll * kThreads;
  constexpr int HPW = 32 / LPH;                             // heads a warp holds per chunk row
  const long n_chunks = n_rows * LPH;                       // (a multiple of LPH: a head is live or dead as a whole)
  const int lane = threadIdx.x & 31;
  const int lane_in_head = lane % LPH;
  for (long tile0 = (long)blockIdx.x * TILE; tile0 < n_chunks; tile0 += (long)gridDim.x * TILE) {
    uint4 raw[kUnroll];
    float m[kUnroll];
#pragma unroll
    for (int k = 0; k < kUnroll; ++k) {
      const long chunk = tile0 + k * kThreads + threadIdx.x;
      raw[k] = chunk < n_chunks ? __ldg(x + chunk) : make_uint4(0, 0, 0, 0);
    }
    // ---- per-head maximum of |x| (on bf16 pairs), shared by the head's lanes ----
#pragma unroll
    for (int k = 0; k < kUnroll; ++k) {
      const uint32_t w[4] = {raw[k].x, raw[k].y, raw[k].z, raw[k].w};
      uint32_t m2 = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t a = w[i] & 0x7FFF7FFFu;
        const __nv_bfloat162 h = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&m2), *reinterpret_cast<const __nv_bfloat162*>(&a));
        m2 = *reinterpret_cast<const uint32_t*>(&h);
      }
      float v = fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xFFFF0000u));
#pragma unroll
      for (int o = LPH / 2; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
      m[k] = v;
    }
    // ---- lane j < kUnroll * HPW takes head (k = j / HPW, h = j % HPW): both divisions, and the scale store ----
    float g = 0.f;
#pragma unroll
    for (int k = 0; k < kUnroll; ++k) {
      const float t = __shfl_sync(0xffffffffu, m[k], (lane % HPW) * LPH);
      if (lane / HPW == k) g = t;
    }
    const float rq_mine = __fdiv_rn((float)(HALF - 1), __fadd_rn(g, eps));
    if (lane < kUnroll * HPW) {
      const long chunk = tile0 + (lane / HPW) * kThreads + (threadIdx.x & ~31) + (lane % HPW) * LPH;
      if (chunk < n_chunks) scale[chunk / LPH] = __fdiv_rn(g, (float)(HALF - 1));
    }
    // ---- quantize and pack ----
#pragma unroll
    for (int k = 0; k < kUnroll; ++k) {
      const long chunk = tile0 + k * kThreads + threadIdx.x;
      const bool live = chunk < n_chunks;
      const long row = (live ? chunk : n_chunks - 1) / LPH;
      const float rq = __shfl_sync(0xffffffffu, rq_mine, k * HPW + lane / LPH);
      float f[8];
      widen8(raw[k], f);
      uint32_t u[8];
      codes8<BITS>(f, rq, u);
      const uint32_t b0 = low_bytes(u[0], u[1], u[2], u[3]), b1 = low_bytes(u[4], u[5], u[6], u[7]);   // codes as bytes
      unsigned char* dst = codes + row * ROW_BYTES;
      if constexpr (BITS == 8) {
        if (live) *reinterpret_cast<uint2*>(dst + 8 * lane_in_head) = make_uint2(b0, b1);
      } else if constexpr (BITS == 4) {
        // byte pairs to nibble pairs: (x | x >> 4) has code 0 | code 1 << 4 in byte 0 and code 2 | code 3 << 4 in byte 2
        const uint32_t o = __byte_perm(b0 | (b0 >> 4), b1 | (b1 >> 4), 0x6420);
        if (live) *reinterpret_cast<uint32_t*>(dst + 4 * lane_in_head) = o;
      } else {
        // 3 bits: 24 bits per lane; four neighbouring lanes make three 32-bit words
        uint32_t o = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) o |= (((b0 >> (8 * i)) & 7u) << (3 * i)) | (((b1 >> (8 * i)) & 7u) << (3 * i + 12));
        const uint32_t next = __shfl_down_sync(0xffffffffu, o, 1);
        const int r = lane_in_head & 3;
        const uint32_t word = r == 0 ? (o | (next << 24)) : r == 1 ? ((o >> 8) | (next << 16)) : ((o >> 16) | (next << 8));
        if (live && r < 3) *reinterpret_cast<uint32_t*>(dst + 12 * (lane_in_head >> 2) + 4 * r) = word;
      }
      // the heads of a [BOS] token are kept at 8 bits as well
      if (bos_codes != nullptr && live) {
        const long token = row / n_heads;
        if (token % seq_len == 0) {
          const long brow = (token / seq_len) * n_heads + row % n_heads;
          uint32_t u8[8];
          codes8<8>(f, __fdiv_rn(127.0f, __fadd_rn(m[k], eps)), u8);
          const uint2 o = make_uint2(low_bytes(u8[0], u8[1], u8[2], u8[3]), low_bytes(u8[4], u8[5], u8[6], u8[7]));
          *reinterpret_cast<uint2*>(bos_codes + brow * (8 * LPH) + 8 * lane_in_head) = o;
          if (lane_in_head == 0) bos_scale[brow] = __fdiv_rn(m[k], 127.0f);
        }
      }
    }
  }
}

template <int BITS, int LPH>
int launch_lph(const void* x, long n_rows, int n_heads, int seq_len, float eps, void* codes, float* scale, void* bos_codes,
               float* bos_scale, cudaStream_t s) {
  const long n_chunks = n_rows * LPH;
  long blocks = (n_chunks + kUnroll * kThreads - 1) / (kUnroll * kThreads);
  const long cap = (long)sm_count() * 32;                   // several waves' worth; beyond that the grid strides
  const int grid = (int)(blocks < cap ? blocks : cap);
  profile_before(KERNEL_ACT, s);
  kv_quant_kernel<BITS, LPH><<<grid, kThreads, 0, s>>>(static_cast<const uint4*>(x), n_rows, n_heads, seq_len, eps,
                                                      static_cast<unsigned char*>(codes), scale,
                                                      static_cast<unsigned char*>(bos_codes), bos_scale);
  profile_after(KERNEL_ACT, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

template <int BITS>
int launch_bits(const void* x, long n_rows, int n_heads, int head_dim, int seq_len, float eps, void* codes, float* scale,
                void* bos_codes, float* bos_scale, cudaStream_t s) {
  switch (head_dim) {
    case 64: return launch_lph<BITS, 8>(x, n_rows, n_heads, seq_len, eps, codes, scale, bos_codes, bos_scale, s);
    case 128: return launch_lph<BITS, 16>(x, n_rows, n_heads, seq_len, eps, codes, scale, bos_codes, bos_scale, s);
    case 256: return launch_lph<BITS, 32>(x, n_rows, n_heads, seq_len, eps, codes, scale, bos_codes, bos_scale, s);
    default: return HBL_ERR_SHAPE;
  }
}

}  // namespace

int launch_kv_quant(const void* x, long n_rows, int n_heads, int head_dim, int bits, int seq_len, float eps, void* codes,
                    float* scale, void* bos_codes, float* bos_scale, cudaStream_t s) {
  if (n_rows <= 0) return HBL_OK;
  switch (bits) {
    case 3: return launch_bits<3>(x, n_rows, n_heads, head_dim, seq_len, eps, codes, scale, bos_codes, bos_scale, s);
    case 4: return launch_bits<4>(x, n_rows, n_heads, head_dim, seq_len, eps, codes, scale, bos_codes, bos_scale, s);
    case 8: return launch_bits<8>(x, n_rows, n_heads, head_dim, seq_len, eps, codes, scale, bos_codes, bos_scale, s);
    default: return HBL_ERR_BITS;
  }
}

}  // namespace hbl
