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
#include <type_traits>

#include "hbl_common.cuh"

namespace hbl {
namespace {

constexpr int kReduceThreads = 256;
constexpr int kMaxPartials = 2048;

// Sum of |w| over one 16-byte vector (four fp32 or eight bf16 values), each term exact in fp64.
template <bool BF16>
__device__ __forceinline__ double abs_sum16(const uint4 v) {
  if constexpr (BF16) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    double t = 0.0;
#pragma unroll
    for (int i = 0; i < 4; ++i)
      t += (double)fabsf(__uint_as_float(w[i] << 16)) + (double)fabsf(__uint_as_float(w[i] & 0xFFFF0000u));
    return t;
  } else {
    return ((double)fabsf(__uint_as_float(v.x)) + (double)fabsf(__uint_as_float(v.y))) +
           ((double)fabsf(__uint_as_float(v.z)) + (double)fabsf(__uint_as_float(v.w)));
  }
}

// Pass 1: fp64 partial sums of |W|, one per CTA, in a fixed order.  `vectors` = the tensor's size in 16-byte
// units; four independent loads per thread are in flight at a time.
template <bool BF16>
__global__ void __launch_bounds__(kReduceThreads)
absmean_partial_kernel(const uint4* __restrict__ W, size_t vectors, double* __restrict__ partials) {
  __shared__ double red[kReduceThreads / 32];
  const size_t per_cta = (vectors + gridDim.x - 1) / gridDim.x;
  const size_t g0 = (size_t)blockIdx.x * per_cta;
  const size_t g1 = min(g0 + per_cta, vectors);
  double acc0 = 0.0, acc1 = 0.0;
  size_t g = g0 + threadIdx.x;
  for (; g + 3 * kReduceThreads < g1; g += 4 * kReduceThreads) {
    const uint4 a = __ldg(W + g), b = __ldg(W + g + kReduceThreads);
    const uint4 c = __ldg(W + g + 2 * kReduceThreads), d = __ldg(W + g + 3 * kReduceThreads);
    acc0 += abs_sum16<BF16>(a) + abs_sum16<BF16>(b);
    acc1 += abs_sum16<BF16>(c) + abs_sum16<BF16>(d);
  }
  for (; g < g1; g += kReduceThreads) acc0 += abs_sum16<BF16>(__ldg(W + g));
  double acc = acc0 + acc1;
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < kReduceThreads / 32; ++w) t += red[w];
    partials[blockIdx.x] = t;
  }
}

// u = w_t + 1 (0, 1, 2) for four consecutive weights, as four bytes.  half_d = (alpha + eps) / 2.
//   fp32: per weight two comparisons, each steering one add of a byte-lane constant.
//   bf16: a bf16 value exceeds the fp32 threshold exactly when it exceeds the threshold truncated to bf16, so
//         the comparisons run on pairs (one instruction per pair and side) and a byte permute lines the four
//         results up.  The "below" side is the unordered comparison: a NaN counts as below, as for fp32.
struct Ternary {
  float half_d;
  __nv_bfloat162 hi2, lo2;
  __device__ explicit Ternary(float h) : half_d(h) {
    const __nv_bfloat16 t = __ushort_as_bfloat16((unsigned short)(__float_as_uint(h) >> 16));
    hi2 = __halves2bfloat162(t, t);
    lo2 = __hneg2(hi2);
  }
  __device__ __forceinline__ uint32_t four(const float4 w) const {
    const float f[4] = {w.x, w.y, w.z, w.w};
    uint32_t u = 0x01010101u;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      if (f[b] > half_d) u += 1u << (8 * b);
      if (!(f[b] >= -half_d)) u -= 1u << (8 * b);
    }
    return u;
  }
  __device__ __forceinline__ uint32_t four(const uint2 w) const {
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&w.x), b = *reinterpret_cast<const __nv_bfloat162*>(&w.y);
    const uint32_t gt = __byte_perm(__hgt2_mask(a, hi2), __hgt2_mask(b, hi2), 0x6420);
    const uint32_t lt = __byte_perm(__hltu2_mask(a, lo2), __hltu2_mask(b, lo2), 0x6420);
    return 0x01010101u + (gt & 0x01010101u) - (lt & 0x01010101u);
  }
};

// Pass 2: every CTA re-derives alpha from the partials (a fixed tree: the same value in every CTA), then
// ternarises and packs.
//
// RoundClip(w / d, -1, 1) with round-half-to-even and d = alpha + eps needs no division: the result is
// sign(w) exactly when fl(|w| / d) > 1/2, and that holds exactly when |w| > d / 2.  (d / 2 is exact in fp32;
// |w| <= d/2 gives a quotient <= 1/2, which rounds to 0; the next fp32 value above d/2 is already more than
// d/2 (1 + 2^-24), whose quotient lies above the midpoint between 1/2 and the next fp32 value, so it rounds
// above 1/2 and then to 1.)  A NaN weight becomes -1, which is what fmin(fmax(rint(NaN), -1), 1) gives.
//
// A warp takes a group of rows of one 128 x 128 tile at a time, 64 bytes per lane in four 16-byte loads.
//   fp32: four rows; lane l loads columns 4l .. 4l+3 of each (one coalesced 512-byte request per row): byte
//         lanes b = 0..3 at bit pair i = l & 3 of packed word l >> 2.  Three shuffles OR the four lanes' parts
//         of a word together and leave lane l with the finished word of row 2 (l & 1) + ((l >> 1) & 1): the
//         warp stores two 64-byte runs.
//   bf16: eight rows; a load takes two rows, lane l columns 8 (l & 15) .. +7 of row l >> 4: bit pairs
//         2 (l & 1) and 2 (l & 1) + 1 of word (l & 15) >> 1.  Two shuffles leave each lane with two finished
//         words.
// The loads of the next group are issued before the current one is packed.
template <bool BF16>
__global__ void __launch_bounds__(256, 4)
ternarise_pack_kernel(const void* __restrict__ W, int N, int K, float eps,
                      const double* __restrict__ partials, int n_partials,
                      uint32_t* __restrict__ packed, float* __restrict__ alpha_out) {
  __shared__ double red[8];
  __shared__ float s_alpha;
  {
    constexpr int PER = kMaxPartials / 256;
    double t = 0.0;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int j = i * 256 + threadIdx.x;
      t += j < n_partials ? partials[j] : 0.0;
    }
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
      double a = 0.0;
      for (int w = 0; w < 8; ++w) a += red[w];
      const float af = (float)(a / ((double)N * (double)K));
      s_alpha = af;
      if (blockIdx.x == 0) *alpha_out = af;
    }
    __syncthreads();
  }
  const Ternary tern(0.5f * (s_alpha + eps));
  const int lane = threadIdx.x & 31;
  const int n_kb = K / 128;
  constexpr int ROWS = BF16 ? 8 : 4;                                // rows per group
  constexpr int GPT = 128 / ROWS;                                   // groups per tile
  const size_t n_groups = (size_t)((N + 127) / 128) * n_kb * GPT;    // (row block, row group, column block)
  const size_t warps = (size_t)gridDim.x * 8;
  const bool b0 = lane & 1, b1 = lane & 2;
  // where this lane's loads start and its finished word(s) go, relative to the group
  const int ld_row = BF16 ? lane >> 4 : 0, ld_vec = BF16 ? lane & 15 : lane;
  const int word = BF16 ? (lane & 15) >> 1 : lane >> 2;             // h = word >> 2, v = word & 3
  const int st_row = BF16 ? 4 * (int)b0 + (lane >> 4) : 2 * (int)b0 + (int)b1;
  const int st_off = (word >> 2) * 512 + st_row * 4 + (word & 3);
  const int shift = BF16 ? 4 * (lane & 1) : 2 * (lane & 3);
  // A group is (rg, kb): row group over the whole tensor, column block; kb runs fastest.  The warp's position
  // and its stride are kept as such pairs, so the loop divides nothing.
  struct Pos { size_t g, rg; int kb; };
  struct Turn { uint4 w[4]; size_t dst; bool inside; };
  const size_t turn_rg = warps / n_kb;
  const int turn_kb = (int)(warps % n_kb);
  auto advance = [&](const Pos p) {
    Pos n = {p.g + warps, p.rg + turn_rg, p.kb + turn_kb};
    if (n.kb >= n_kb) { n.kb -= n_kb; ++n.rg; }
    return n;
  };
  // No branch in fetch or emit: a group of padding rows (and a position past the end, fetched once before the
  // loop stops) loads the tensor's last row instead and the result is replaced afterwards.
  auto fetch = [&](const Pos p, Turn& u) {
    const int rb = (int)(p.rg / GPT), r0 = (int)(p.rg % GPT) * ROWS;
    const int R = rb * 128 + r0;
    u.inside = R < N;                                               // N % 16 == 0: a group is inside or outside
    u.dst = ((size_t)rb * n_kb + p.kb) * 1024 + (size_t)r0 * 4 + st_off;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int row = min(R + (BF16 ? 2 * j : j) + ld_row, N - 1);
      u.w[j] = __ldg(reinterpret_cast<const uint4*>(W) + (((size_t)row * K + (size_t)p.kb * 128) >> (BF16 ? 3 : 2)) + ld_vec);
    }
  };
  auto emit = [&](const Turn& u) {
    uint32_t p[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if constexpr (BF16)
        p[j] = (tern.four(make_uint2(u.w[j].x, u.w[j].y)) | (tern.four(make_uint2(u.w[j].z, u.w[j].w)) << 2)) << shift;
      else
        p[j] = tern.four(make_float4(__uint_as_float(u.w[j].x), __uint_as_float(u.w[j].y), __uint_as_float(u.w[j].z),
                                     __uint_as_float(u.w[j].w))) << shift;
    }
    uint32_t k0 = b0 ? p[2] : p[0], k1 = b0 ? p[3] : p[1];
    k0 |= __shfl_xor_sync(0xffffffffu, b0 ? p[0] : p[2], 1);
    k1 |= __shfl_xor_sync(0xffffffffu, b0 ? p[1] : p[3], 1);
    if constexpr (!BF16) k0 = (b1 ? k1 : k0) | __shfl_xor_sync(0xffffffffu, b1 ? k0 : k1, 2);
    packed[u.dst] = u.inside ? k0 : 0x55555555u;                    // padding rows: w = 0
    if constexpr (BF16) packed[u.dst + 8] = u.inside ? k1 : 0x55555555u;   // two rows further down
  };
  const size_t g_first = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  Pos pos = {g_first, g_first / n_kb, (int)(g_first % n_kb)};
  if (pos.g >= n_groups) return;
  Turn a, b;
  fetch(pos, a);
  for (;;) {
    pos = advance(pos);
    fetch(pos, b);
    emit(a);
    if (pos.g >= n_groups) break;
    pos = advance(pos);
    fetch(pos, a);
    emit(b);
    if (pos.g >= n_groups) break;
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
  const bool bf16 = w_dtype == HBL_BF16;
  const size_t vectors = total / (bf16 ? 8 : 4);
  if (bf16) absmean_partial_kernel<true><<<grid, kReduceThreads, 0, s>>>(static_cast<const uint4*>(W), vectors, partials);
  else absmean_partial_kernel<false><<<grid, kReduceThreads, 0, s>>>(static_cast<const uint4*>(W), vectors, partials);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  const size_t n_groups = (size_t)((N + 127) / 128) * (K / 128) * (bf16 ? 16 : 32);
  int grid2 = (int)min((size_t)148 * 4, (n_groups + 7) / 8);      // one resident wave: 4 thread blocks of 256 per SM
  if (bf16) ternarise_pack_kernel<true><<<grid2, 256, 0, s>>>(W, N, K, eps, partials, grid, static_cast<uint32_t*>(packed), alpha);
  else ternarise_pack_kernel<false><<<grid2, 256, 0, s>>>(W, N, K, eps, partials, grid, static_cast<uint32_t*>(packed), alpha);
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
