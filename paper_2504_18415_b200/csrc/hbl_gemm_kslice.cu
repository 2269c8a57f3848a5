// Small-batch contraction of H-BitLinear (Eq. 7) for T <= 32 tokens, bound by the
// stream of 2-bit packed weights out of HBM.
//
// Persistent, one CTA per SM: a producer thread keeps a deep shared-memory ring
// (up to 160 KiB) full with bulk async copies of packed weights, so the HBM pipe
// never drains, and eight consumer warps contract what arrives.
//
// The K axis is sliced over the consumer warps: warp w owns KW columns of every
// "pass" of P = 8*KW columns and keeps the tokens' int8 codes for its slice in
// registers as m16n8k32 B fragments for as long as the pass lasts.  Weights
// therefore cross shared memory exactly once (ring in, 128-bit fragment loads out)
// and the codes never do; what does cross it is the reduction of the eight warps'
// partial sums, 16 T / KW bytes per weight byte.
//
// Work is counted in quanta of one 512-byte tile per warp (8 tiles, 4 KiB, per
// quantum), ordered [16-row tile][pass][tile], and dealt to the CTAs as equal
// contiguous ranges: every SM streams the same number of bytes whatever N and K
// are.  A row tile whose quanta straddle two CTAs is finished by the CTA that
// holds its head: the CTA that holds the tail adds its part into a scratch slot of
// its own, raises a flag, and the head's CTA, when its range is done, picks the
// part up (a bounded wait on a flag that was raised long before) and runs the
// epilogue.  Integer sums: the result does not depend on who adds what.
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

constexpr int MAX_STAGES = 32;

template <int KW>
struct Shape {
  static constexpr int P = CW * KW;                   // columns per pass
  static constexpr int UNIT_BYTES = 4 * P;            // 16 rows x P columns x 2 bits: one ring stage
  static constexpr int TILES = KW / 128;              // 512-byte tiles per warp per (row tile, pass)
};

// One work item: the tiles [ta, tb) of every warp for (row tile rt, pass).
struct Item { int rt, pass, ta, tb; };

// The CTA's range [q0, q1) of quanta, ordered [rt][pass][tile], walked pass-major so that the
// code fragments are reloaded once per pass.  Producer and consumers run the same walk.
template <int TILES>
struct Walk {
  long q0, q1;
  int n_pass, rt_first, rt_last;
  int pass, rt;
  __device__ Walk(long q0_, long q1_, int n_pass_) : q0(q0_), q1(q1_), n_pass(n_pass_) {
    const long per_rt = (long)n_pass * TILES;
    rt_first = (int)(q0 / per_rt);
    rt_last = (int)((q1 - 1) / per_rt);
    pass = 0;
    rt = rt_first - 1;
  }
  __device__ bool next(Item& it) {
    while (pass < n_pass) {
      while (++rt <= rt_last) {
        const long base = ((long)rt * n_pass + pass) * TILES;
        const long a = q0 > base ? q0 - base : 0, b = (q1 - base) < TILES ? (q1 - base) : TILES;
        if (a < b) { it.rt = rt; it.pass = pass; it.ta = (int)a; it.tb = (int)b; return true; }
      }
      ++pass;
      rt = rt_first - 1;
    }
    return false;
  }
};

struct Params {
  const int8_t* codes; const float* scale; const int32_t* codesum;
  const unsigned char* Wp; const float* alpha;
  __nv_bfloat16* y; int32_t* acc_out;
  int32_t* part;      // [grid][128*NT] partial sums of row tiles shared with the previous CTA
  int* flags;         // [grid], zero on entry: flags[c] = 1 once part[c] is complete
  int* status;
  int T, K, N;
  int stages;         // ring depth (host-chosen so that everything fits in shared memory)
  int acc_tiles;      // row tiles of shared-memory accumulators (0 when K is a single pass)
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
  constexpr int TILES = S::TILES;
  constexpr int SLOTS = 128 * NT;                      // outputs of one row tile: 16 rows x 8*NT tokens
  constexpr int VPT = (SLOTS + CONSUMERS - 1) / CONSUMERS;   // outputs per consumer thread
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* ring = smem;
  int* red = reinterpret_cast<int*>(smem + (size_t)p.stages * S::UNIT_BYTES);   // [2][CW][SLOTS]
  int* acc_sm = red + 2 * CW * SLOTS;                  // [acc_tiles][SLOTS] sums over passes
  int* tail_sm = acc_sm + (size_t)p.acc_tiles * SLOTS; // [SLOTS] this CTA's part of its last, shared row tile
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ int abort_flag_s;
  __shared__ int s_abort_seen;                         // set-only; read after the reduction barrier so that all warps agree
  __shared__ int s_part_ready;
  volatile int* abort_flag = &abort_flag_s;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int stages = p.stages;
  const int n_rt = p.N / 16, n_pass = p.K / S::P;
  const long per_rt = (long)n_pass * TILES;
  const long Q = (long)n_rt * per_rt;
  const long q0 = Q * blockIdx.x / gridDim.x, q1 = Q * (blockIdx.x + 1) / gridDim.x;
  const bool head_shared = (q0 % per_rt) != 0;         // my first row tile begins in the previous CTA
  const bool tail_shared = (q1 % per_rt) != 0;         // my last row tile ends in the next CTA

  if (tid == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], CW); }
    abort_flag_s = 0;
    s_abort_seen = 0;
    s_part_ready = 0;
    mbar_fence_init();
  }
  __syncthreads();

  if (warp == CW) {
    // ------------------------------ producer ------------------------------
    if (lane == 0 && q1 > q0) {
      Walk<TILES> walk(q0, q1, n_pass);
      Item it;
      for (int i = 0; walk.next(it); ++i) {
        const int s = i % stages;
        if (!mbar_wait(&empty_bar[s], ((i / stages) & 1) ^ 1, abort_flag, p.status)) break;
        const unsigned char* src = p.Wp + ((size_t)it.rt * (p.K / 128) + (size_t)it.pass * (S::P / 128)) * 512;
        unsigned char* dst = ring + (size_t)s * S::UNIT_BYTES;
        const int nt = it.tb - it.ta;
        mbar_expect_tx(&full_bar[s], (uint32_t)(CW * nt * 512));
        if (nt == TILES) {
          bulk_load(dst, src, S::UNIT_BYTES, &full_bar[s]);
        } else {
          for (int w = 0; w < CW; ++w)
            bulk_load(dst + (size_t)(w * TILES + it.ta) * 512, src + (size_t)(w * TILES + it.ta) * 512,
                      (uint32_t)(nt * 512), &full_bar[s]);
        }
      }
    }
  } else if (q1 > q0) {
    // ------------------------------ consumers ------------------------------
    const int g = lane >> 2, t4 = lane & 3;
    const float al = (p.acc_out == nullptr) ? __ldg(p.alpha) : 0.f;
    Walk<TILES> walk(q0, q1, n_pass);
    const int rt_first = walk.rt_first, rt_last = walk.rt_last;
    const int last_pass_of_tail = (int)(((q1 - 1) % per_rt) / TILES);
    if (p.acc_tiles > 0) {
      for (int i = tid; i < p.acc_tiles * SLOTS; i += CONSUMERS) acc_sm[i] = 0;   // thread-owned slots: no barrier needed
    }
    uint32_t bfrag[KW / 32][NT][2];
    int cur_pass = -1;
    bool ok = true;
    Item it;
    for (int i = 0; walk.next(it); ++i) {
      const int s = i % stages;
      if (it.pass != cur_pass) {
        // the tokens' codes for this warp's slice of the pass, as B fragments, straight from global memory
        cur_pass = it.pass;
        const int8_t* base = p.codes + (size_t)it.pass * S::P + warp * KW + 4 * t4;
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
      ok = ok && mbar_wait(&full_bar[s], (i / stages) & 1, abort_flag, p.status);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        const uint4* tiles =
            reinterpret_cast<const uint4*>(ring + (size_t)s * S::UNIT_BYTES + (size_t)warp * TILES * 512) + lane;
        uint4 w[TILES];
#pragma unroll
        for (int t = 0; t < TILES; ++t) w[t] = (t >= it.ta && t < it.tb) ? tiles[t * 32] : make_uint4(0, 0, 0, 0);
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[s]);          // the stage is in registers: hand it back
#pragma unroll
        for (int t = 0; t < TILES; ++t) {
          if (t < it.ta || t >= it.tb) continue;            // uniform over the CTA
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
      // ---- reduce the eight warps' partial sums (double-buffered: one barrier per item) ----
      int* rbuf = red + (size_t)(i & 1) * CW * SLOTS;
#pragma unroll
      for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int q = 0; q < 4; ++q) rbuf[warp * SLOTS + (n * 4 + q) * 32 + lane] = acc[n][q];
      if (!ok && lane == 0) s_abort_seen = 1;
      named_barrier(1, CONSUMERS);
      if (*(volatile int*)&s_abort_seen) continue;          // aborted: keep meeting barrier 1, do no work
      const int lr = it.rt - rt_first;
      const bool complete = it.pass == ((it.rt == rt_last) ? last_pass_of_tail : n_pass - 1);   // my last item of this row tile
      const bool is_head_part = head_shared && it.rt == rt_first;   // the tile's head lives in the previous CTA
      const bool is_tail_part = tail_shared && it.rt == rt_last;    // the tile's tail lives in the next CTA
#pragma unroll
      for (int r = 0; r < VPT; ++r) {
        const int slot = tid + r * CONSUMERS;
        if (slot >= SLOTS) continue;
        int v = 0;
#pragma unroll
        for (int w8 = 0; w8 < CW; ++w8) v += rbuf[w8 * SLOTS + slot];
        if (p.acc_tiles > 0) {
          v += acc_sm[lr * SLOTS + slot];
          acc_sm[lr * SLOTS + slot] = v;
        }
        if (!complete) continue;
        if (is_head_part) {
          __stcg(p.part + (size_t)blockIdx.x * SLOTS + slot, v);
        } else if (is_tail_part) {
          tail_sm[slot] = v;
        } else {
          int tok, row;
          slot_coords(slot, it.rt, tok, row);
          if (tok < p.T) finish(p, tok, row, v, al);
        }
      }
      if (complete && is_head_part) {                       // uniform over the consumers
        __threadfence();
        named_barrier(2, CONSUMERS);
        if (tid == 0) atomicExch(p.flags + blockIdx.x, 1);
      }
    }
    // ---- my last row tile continues in the next CTA: fetch its part (published early in its run) ----
    if (tail_shared && !*(volatile int*)&s_abort_seen) {
      if (tid == 0) {
        volatile int* flag = p.flags + blockIdx.x + 1;
        const uint64_t t0 = global_ns();
        int ready = 0;
        while (!(ready = *flag)) {
          if (*abort_flag) break;
          if (global_ns() - t0 > 2000000000ull) {
            report_device_error(p.status, HBL_ERR_TIMEOUT);
            *abort_flag = 1;
            break;
          }
          __nanosleep(100);
        }
        s_part_ready = ready;
      }
      named_barrier(2, CONSUMERS);
      if (s_part_ready) {
        __threadfence();
#pragma unroll
        for (int r = 0; r < VPT; ++r) {
          const int slot = tid + r * CONSUMERS;
          if (slot >= SLOTS) continue;
          const int v = tail_sm[slot] + __ldcg(p.part + (size_t)(blockIdx.x + 1) * SLOTS + slot);
          int tok, row;
          slot_coords(slot, rt_last, tok, row);
          if (tok < p.T) finish(p, tok, row, v, al);
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

// Host-side plan of one launch.
struct Plan {
  int nt, kw, n_pass, grid, stages, acc_tiles;
  size_t smem;
};

constexpr size_t kSmemBudget = 226 * 1024;   // dynamic shared memory the kernel may ask for (227 KiB per CTA minus its static part)

bool make_plan(int T, int K, int N, Plan* pl) {
  if (T < 1 || T > 32 || K % (CW * 128) != 0 || N % 16 != 0) return false;
  pl->nt = T <= 8 ? 1 : (T <= 16 ? 2 : 4);
  // the widest slice whose code fragments fit in 64 registers (KW * NT <= 1024) and that divides K
  pl->kw = 0;
  const int cands[4] = {1024, 512, 256, 128};
  for (int i = 0; i < 4 && pl->kw == 0; ++i)
    if (cands[i] * pl->nt <= 1024 && K % (CW * cands[i]) == 0) pl->kw = cands[i];
  if (pl->kw == 0) return false;
  pl->n_pass = K / (CW * pl->kw);
  const int n_rt = N / 16, n_sm = sm_count();
  pl->grid = n_rt < n_sm ? n_rt : n_sm;      // every CTA gets at least one whole row tile's worth of quanta
  const size_t slots = 128 * (size_t)pl->nt;
  pl->acc_tiles = pl->n_pass > 1 ? (n_rt + pl->grid - 1) / pl->grid + 2 : 0;
  const size_t fixed = sizeof(int) * slots * (2 * CW + (size_t)pl->acc_tiles + 1);
  const size_t unit = 32 * (size_t)pl->kw;
  if (fixed + 2 * unit > kSmemBudget) return false;
  size_t ring = kSmemBudget - fixed;
  if (ring > (size_t)RING_BYTES) ring = RING_BYTES;
  pl->stages = (int)(ring / unit);
  if (pl->stages > MAX_STAGES) pl->stages = MAX_STAGES;
  pl->smem = (size_t)pl->stages * unit + fixed;
  return true;
}

template <int NT, int KW>
int launch_variant(const Params& p, const Plan& pl, cudaStream_t s) {
  auto kern = gemm_kslice_kernel<NT, KW>;
  static bool done = false;   // idempotent attribute; a race only repeats the call
  if (!done) {
    HBL_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBudget));
    done = true;
  }
  profile_before(KERNEL_CONTRACT, s);
  kern<<<pl.grid, THREADS, pl.smem, s>>>(p);
  profile_after(KERNEL_CONTRACT, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

}  // namespace

bool gemm_kslice_supported(int T, int K, int N) {
  Plan pl;
  return make_plan(T, K, N, &pl);
}

// Number of flag words (from the start of `flags`) that must be zero on entry.
int gemm_kslice_flag_words(int T, int K, int N) {
  Plan pl;
  return make_plan(T, K, N, &pl) ? pl.grid : 0;
}

// part: at least grid * 128 * NT int32 words (contents irrelevant); flags: grid words, zero on entry.
int launch_gemm_kslice(const int8_t* codes, const float* scale, const int32_t* codesum, int T, int K,
                       const void* W_packed, int N, const float* alpha, __nv_bfloat16* y, int32_t* acc_out,
                       int32_t* part, int* flags, cudaStream_t s) {
  if (T <= 0) return HBL_OK;
  Plan pl;
  if (!make_plan(T, K, N, &pl)) return HBL_ERR_SHAPE;
  Params p;
  p.codes = codes; p.scale = scale; p.codesum = codesum; p.Wp = static_cast<const unsigned char*>(W_packed);
  p.alpha = alpha; p.y = y; p.acc_out = acc_out; p.part = part; p.flags = flags;
  p.status = device_status_word();
  if (p.status == nullptr) return HBL_ERR_CUDA;
  p.T = T; p.K = K; p.N = N; p.stages = pl.stages; p.acc_tiles = pl.acc_tiles;
#define HBL_V(NT_, KW_) if (pl.nt == NT_ && pl.kw == KW_) return launch_variant<NT_, KW_>(p, pl, s);
  HBL_V(1, 1024) HBL_V(1, 512) HBL_V(1, 256) HBL_V(1, 128)
  HBL_V(2, 512) HBL_V(2, 256) HBL_V(2, 128)
  HBL_V(4, 256) HBL_V(4, 128)
#undef HBL_V
  return HBL_ERR_SHAPE;
}

}  // namespace hbl
