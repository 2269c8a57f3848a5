// Small-batch contraction of H-BitLinear (Eq. 7) for T <= 32 tokens, bound by the
// stream of 2-bit packed weights out of HBM.
//
// Persistent, one CTA per SM: a producer thread keeps a deep shared-memory ring
// (~160 KiB) full with bulk async copies of packed weights, so the HBM pipe never
// drains, and eight consumer warps contract what arrives.
//
// The K axis is sliced over the consumer warps: warp w owns KW columns of every
// "pass" of P = 8*KW columns and keeps the tokens' int8 codes for its slice in
// registers as m16n8k32 B fragments for as long as the pass lasts.  Weights
// therefore cross shared memory exactly once (ring in, 128-bit fragment loads out)
// and the codes never do; what does cross it is the reduction of the eight warps'
// partial sums, 16 T / KW bytes per weight byte.
//
// A unit of work is one 16-row tile of W over one pass: 32*KW contiguous bytes of
// the packed tensor.  Units are numbered pass-major and dealt to the CTAs in equal
// contiguous ranges, so a CTA reloads its code fragments at most a few times.
// With more than one pass the per-pass sums are combined with integer atomics in a
// zeroed scratch array (order independent) and the last pass to arrive for a row
// tile runs the epilogue.
//
// Weights are stored as u = w + 1 and fed as unsigned bytes: sum_k u q = sum_k w q + sum_k q;
// the epilogue subtracts the token's code sum.
#include "hbl_pipeline.cuh"

namespace hbl {
namespace {

using namespace pipe;

constexpr int CW = 8;                       // consumer warps
constexpr int CONSUMERS = CW * 32;
constexpr int THREADS = CONSUMERS + 32;     // + the producer warp
constexpr int RING_BYTES = 160 * 1024;

__device__ __forceinline__ void mma_u8s8(int (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int KW>
struct Shape {
  static constexpr int P = CW * KW;                   // columns per pass
  static constexpr int UNIT_BYTES = 4 * P;            // 16 rows x P columns x 2 bits
  static constexpr int TILES = KW / 128;              // 512-byte tiles per warp per unit
  static constexpr int STAGES_RAW = RING_BYTES / UNIT_BYTES;
  static constexpr int STAGES = STAGES_RAW > 32 ? 32 : STAGES_RAW;
};

struct Params {
  const int8_t* codes; const float* scale; const int32_t* codesum;
  const unsigned char* Wp; const float* alpha;
  __nv_bfloat16* y; int32_t* acc_out; int32_t* acc_ws; int* counters; int* status;
  int T, K, N;
};

// Final value of one output: subtract the code sum, then either export the int32 or rescale to bf16.
__device__ __forceinline__ void finish(const Params& p, int tok, int row, int v, float al) {
  const int a = v - __ldg(p.codesum + tok);
  if (p.acc_out != nullptr) p.acc_out[(size_t)tok * p.N + row] = a;
  else p.y[(size_t)tok * p.N + row] = __float2bfloat16_rn((float)a * (__ldg(p.scale + tok) * al));
}

// slot = (n*4 + q)*32 + l  ->  row 16 rt + (l>>2) + 8 (q>>1), token 8n + 2 (l&3) + (q&1)
__device__ __forceinline__ void slot_coords(int slot, int rt, int& tok, int& row) {
  const int l = slot & 31, q = (slot >> 5) & 3, n = slot >> 7;
  tok = 8 * n + 2 * (l & 3) + (q & 1);
  row = 16 * rt + (l >> 2) + 8 * (q >> 1);
}

template <int NT, int KW>
__global__ void __launch_bounds__(THREADS, 1) gemm_kslice_kernel(const Params p) {
  using S = Shape<KW>;
  constexpr int STAGES = S::STAGES;
  constexpr int SLOTS = 128 * NT;                      // outputs of one unit: 16 rows x 8*NT tokens
  constexpr int VPT = (SLOTS + CONSUMERS - 1) / CONSUMERS;   // outputs per consumer thread
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* ring = smem;
  int* red = reinterpret_cast<int*>(smem + (size_t)STAGES * S::UNIT_BYTES);   // [2][CW][SLOTS]
  __shared__ __align__(8) uint64_t full_bar[STAGES];
  __shared__ __align__(8) uint64_t empty_bar[STAGES];
  __shared__ int abort_flag_s;
  __shared__ int s_last;
  __shared__ int s_abort_seen;                         // set-only; read after the reduction barrier so that all warps agree
  volatile int* abort_flag = &abort_flag_s;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_rt = p.N / 16, n_pass = p.K / S::P;
  const long U = (long)n_rt * n_pass;
  const long u0 = U * blockIdx.x / gridDim.x, u1 = U * (blockIdx.x + 1) / gridDim.x;
  const int n_units = (int)(u1 - u0);

  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], CW); }
    abort_flag_s = 0;
    s_abort_seen = 0;
    mbar_fence_init();
  }
  __syncthreads();

  if (warp == CW) {
    // ------------------------------ producer ------------------------------
    if (lane == 0) {
      for (int i = 0; i < n_units; ++i) {
        const int s = i % STAGES;
        if (!mbar_wait(&empty_bar[s], ((i / STAGES) & 1) ^ 1, abort_flag, p.status)) break;
        const long u = u0 + i;
        const int pass = (int)(u / n_rt), rt = (int)(u % n_rt);
        const unsigned char* src = p.Wp + ((size_t)rt * (p.K / 128) + (size_t)pass * (S::P / 128)) * 512;
        mbar_expect_tx(&full_bar[s], S::UNIT_BYTES);
        bulk_load(ring + (size_t)s * S::UNIT_BYTES, src, S::UNIT_BYTES, &full_bar[s]);
      }
    }
  } else {
    // ------------------------------ consumers ------------------------------
    const int g = lane >> 2, t4 = lane & 3;
    const float al = (p.acc_out == nullptr) ? __ldg(p.alpha) : 0.f;
    uint32_t bfrag[KW / 32][NT][2];
    int cur_pass = -1;
    bool ok = true;
    for (int i = 0; i < n_units; ++i) {
      const int s = i % STAGES;
      const long u = u0 + i;
      const int pass = (int)(u / n_rt), rt = (int)(u % n_rt);
      if (pass != cur_pass) {
        // the tokens' codes for this warp's slice of the pass, as B fragments, straight from global memory
        cur_pass = pass;
        const int8_t* base = p.codes + (size_t)pass * S::P + warp * KW + 4 * t4;
#pragma unroll
        for (int n = 0; n < NT; ++n) {
          const int tok = 8 * n + g;
          const int8_t* row = base + (size_t)tok * p.K;
#pragma unroll
          for (int jj = 0; jj < KW / 32; ++jj) {
            bfrag[jj][n][0] = tok < p.T ? __ldg(reinterpret_cast<const uint32_t*>(row + jj * 32)) : 0u;
            bfrag[jj][n][1] = tok < p.T ? __ldg(reinterpret_cast<const uint32_t*>(row + jj * 32 + 16)) : 0u;
          }
        }
      }
      int acc[NT][4];
#pragma unroll
      for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[n][q] = 0;
      ok = ok && mbar_wait(&full_bar[s], (i / STAGES) & 1, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        const uint4* tiles =
            reinterpret_cast<const uint4*>(ring + (size_t)s * S::UNIT_BYTES + (size_t)warp * S::TILES * 512) + lane;
        uint4 w[S::TILES];
#pragma unroll
        for (int t = 0; t < S::TILES; ++t) w[t] = tiles[t * 32];
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[s]);          // the stage is in registers: hand it back
#pragma unroll
        for (int t = 0; t < S::TILES; ++t) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t word = (j == 0) ? w[t].x : (j == 1) ? w[t].y : (j == 2) ? w[t].z : w[t].w;
            uint32_t a[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) a[q] = (word >> (2 * q)) & 0x03030303u;
#pragma unroll
            for (int n = 0; n < NT; ++n) mma_u8s8(acc[n], a, bfrag[t * 4 + j][n][0], bfrag[t * 4 + j][n][1]);
          }
        }
      }
      // ---- reduce the eight warps' partial sums (double-buffered: one barrier per unit) ----
      int* rbuf = red + (size_t)(i & 1) * CW * SLOTS;
#pragma unroll
      for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int q = 0; q < 4; ++q) rbuf[warp * SLOTS + (n * 4 + q) * 32 + lane] = acc[n][q];
      if (!ok && lane == 0) s_abort_seen = 1;
      named_barrier(1, CONSUMERS);
      if (*(volatile int*)&s_abort_seen) continue;          // aborted: keep meeting barrier 1, do no work
      int v[VPT];
#pragma unroll
      for (int r = 0; r < VPT; ++r) {
        const int slot = tid + r * CONSUMERS;
        int sum = 0;
        if (slot < SLOTS) {
#pragma unroll
          for (int w8 = 0; w8 < CW; ++w8) sum += rbuf[w8 * SLOTS + slot];
        }
        v[r] = sum;
      }
      if (n_pass == 1) {
#pragma unroll
        for (int r = 0; r < VPT; ++r) {
          const int slot = tid + r * CONSUMERS;
          int tok, row;
          slot_coords(slot, rt, tok, row);
          if (slot < SLOTS && tok < p.T) finish(p, tok, row, v[r], al);
        }
      } else {
#pragma unroll
        for (int r = 0; r < VPT; ++r) {
          const int slot = tid + r * CONSUMERS;
          int tok, row;
          slot_coords(slot, rt, tok, row);
          if (slot < SLOTS && tok < p.T) atomicAdd(p.acc_ws + (size_t)tok * p.N + row, v[r]);
        }
        __threadfence();
        named_barrier(2, CONSUMERS);
        if (tid == 0) s_last = (atomicAdd(p.counters + rt, 1) == n_pass - 1);
        named_barrier(2, CONSUMERS);
        if (s_last) {
          __threadfence();
#pragma unroll
          for (int r = 0; r < VPT; ++r) {
            const int slot = tid + r * CONSUMERS;
            int tok, row;
            slot_coords(slot, rt, tok, row);
            if (slot < SLOTS && tok < p.T) finish(p, tok, row, __ldcg(p.acc_ws + (size_t)tok * p.N + row), al);
          }
        }
      }
    }
  }
  // Teardown: nothing may still be writing this CTA's shared memory when it exits.  Normally every
  // issued copy was waited for by the consumers; after an abort give copies in flight time to land.
  __syncthreads();
  if (*abort_flag) {
    const uint64_t t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
  }
}

template <int NT, int KW>
int launch_variant(const Params& p, int grid, cudaStream_t s) {
  using S = Shape<KW>;
  const size_t smem = (size_t)S::STAGES * S::UNIT_BYTES + sizeof(int) * 2 * CW * 128 * NT;
  auto kern = gemm_kslice_kernel<NT, KW>;
  static bool done = false;   // idempotent attribute; a race only repeats the call
  if (!done) {
    HBL_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    done = true;
  }
  profile_before(KERNEL_CONTRACT, s);
  kern<<<grid, THREADS, smem, s>>>(p);
  profile_after(KERNEL_CONTRACT, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = 148;
  }
  return n;
}

int tiles_of_tokens(int T) { return T <= 8 ? 1 : (T <= 16 ? 2 : 4); }

// Slice width: the widest that keeps the chip evenly loaded.  A narrow slice means more
// reduction traffic per weight byte (16 T / KW), so 128 is taken only when it balances much better.
int choose_kw(int nt, int K, int N, int n_sm) {
  const int cands[4] = {1024, 512, 256, 128};
  int best = 0;
  double best_score = -1.0;
  for (int i = 0; i < 4; ++i) {
    const int kw = cands[i];
    if (kw * nt > 1024 || K % (CW * kw) != 0) continue;
    const long U = (long)(N / 16) * (K / (CW * kw));
    const long g = U < n_sm ? U : n_sm;
    const double balance = (double)U / (double)(g * ((U + g - 1) / g));
    const double score = balance * (kw >= 256 ? 1.0 : 0.93);
    if (score > best_score + 0.02) { best_score = score; best = kw; }
  }
  return best;
}

}  // namespace

bool gemm_kslice_supported(int T, int K) { return T >= 1 && T <= 32 && K % (CW * 128) == 0; }

// Number of passes over K the kernel will make for this problem (1 = no scratch is touched).
int gemm_kslice_passes(int T, int K, int N) {
  const int kw = choose_kw(tiles_of_tokens(T), K, N, sm_count());
  return kw == 0 ? 0 : K / (CW * kw);
}

// acc_ws [T*N] and counters [N/16] must be zero on entry when K spans more than one pass.
int launch_gemm_kslice(const int8_t* codes, const float* scale, const int32_t* codesum, int T, int K,
                       const void* W_packed, int N, const float* alpha, __nv_bfloat16* y, int32_t* acc_out,
                       int32_t* acc_ws, int* counters, cudaStream_t s) {
  if (T <= 0) return HBL_OK;
  if (!gemm_kslice_supported(T, K)) return HBL_ERR_SHAPE;
  const int nt = tiles_of_tokens(T);
  const int n_sm = sm_count();
  const int kw = choose_kw(nt, K, N, n_sm);
  if (kw == 0) return HBL_ERR_SHAPE;
  Params p;
  p.codes = codes; p.scale = scale; p.codesum = codesum; p.Wp = static_cast<const unsigned char*>(W_packed);
  p.alpha = alpha; p.y = y; p.acc_out = acc_out; p.acc_ws = acc_ws; p.counters = counters;
  p.status = device_status_word();
  if (p.status == nullptr) return HBL_ERR_CUDA;
  p.T = T; p.K = K; p.N = N;
  const long U = (long)(N / 16) * (K / (CW * kw));
  const int grid = (int)(U < n_sm ? U : n_sm);
#define HBL_V(NT_, KW_) if (nt == NT_ && kw == KW_) return launch_variant<NT_, KW_>(p, grid, s);
  HBL_V(1, 1024) HBL_V(1, 512) HBL_V(1, 256) HBL_V(1, 128)
  HBL_V(2, 512) HBL_V(2, 256) HBL_V(2, 128)
  HBL_V(4, 256) HBL_V(4, 128)
#undef HBL_V
  return HBL_ERR_SHAPE;
}

}  // namespace hbl
