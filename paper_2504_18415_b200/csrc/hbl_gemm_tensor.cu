// Large-batch contraction of H-BitLinear (Eq. 7) on the 5th-generation tensor
// cores: tcgen05.mma kind::i8 (int8 x int8 -> int32) with the accumulators in
// tensor memory, operands staged in shared memory by TMA, and the epilogue
// (alpha * s_t rescale, one rounding to bf16) reading the accumulators back with
// tcgen05.ld.
//
//   D[128 tokens, 256 weight rows] += A[128, 32] * B[256, 32]^T   per instruction
//   (128 weight rows per tile on very small grids, see launch_gemm_tensor)
//
// Persistent, warp-specialised, one CTA per SM:
//   warp 0      TMA producer: 4-stage ring of (A 128x128 B, B 256x128 B) tiles, 128-byte swizzle
//   warp 1      allocates the 512 TMEM columns, one lane issues the MMAs and commits
//   warps 2..5  epilogue: each owns the TMEM lane quadrant (warp & 3)
// Two 256-column accumulators alternate so that the epilogue of tile i overlaps
// the main loop of tile i+1.
//
// Every wait is bounded: when a barrier does not flip within ~2 s the waiting
// thread records HBL_ERR_TIMEOUT in the status word and raises a CTA-wide abort
// flag that all roles poll; the CTA then drains, frees its tensor memory and
// returns.  No TMA multicast is used anywhere.
#include <cuda.h>

#include "hbl_pipeline.cuh"

namespace hbl {
namespace {

using namespace pipe;   // bounded mbarrier waits

constexpr int BM = 128;              // tokens per tile (MMA M, TMEM lanes)
constexpr int BK = 128;              // bytes (= int8 elements) of K per stage: one swizzle atom
constexpr int UMMA_K = 32;           // K of one kind::i8 instruction
constexpr int A_BYTES = BM * BK;     // 16 KiB
constexpr int THREADS = 192;
constexpr int TMEM_COLS = 512;
// Weight rows per tile (MMA N, TMEM columns): 256 is the efficient shape; 128 is used when 256-row tiles
// would leave half of the SMs without a tile (it doubles the number of tiles).
// PACKED: the tokens' INT4 codes arrive two per byte (Eq. 6's codes, packed by the activation kernel).  Each
// stage then also holds the 8 KiB packed tile as TMA delivers it, and eight more warps widen it into the int8
// token tile the tensor cores read.
constexpr int PK_BYTES = BM * BK / 2;                    // packed token tile of one stage: 128 rows x 64 bytes
constexpr int WIDEN_THREADS = 256;                       // two threads per token row of the tile
template <int BN, bool PACKED = false>
struct Shape {
  static constexpr int STAGES = BN == 256 ? 4 : (PACKED ? 5 : 6);
  static constexpr int B_BYTES = BN * BK;                // 32 or 16 KiB
  static constexpr int TX_BYTES = (PACKED ? PK_BYTES : A_BYTES) + B_BYTES;     // what the copies of one stage deliver
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES + (PACKED ? PK_BYTES : 0);
  static constexpr int N_THREADS = THREADS + (PACKED ? WIDEN_THREADS : 0);
  static constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 1024;   // + alignment slack
  // Instruction descriptor (32 bit): D format s32 (2) at bits [4,6); A and B format
  // signed 8-bit (1) at [7,10) and [10,13); both K-major (bits 15, 16 = 0);
  // N >> 3 at [17,23); M >> 4 at [24,29).
  static constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) |
                                    ((uint32_t)(BM >> 4) << 24);
};
constexpr int MAX_STAGES = 6;


// Shared-memory matrix descriptor, K-major operand in the 128-byte swizzle:
// start address >> 4 at [0,14); leading byte offset (unused for swizzled K-major) = 1 at [16,30);
// stride byte offset = 1024 B between 8-row groups, >> 4, at [32,46); version 1 at [46,48);
// layout type 2 (128-byte swizzle) at [61,64).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  return (uint64_t)((saddr >> 4) & 0x3FFF) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}

__device__ __forceinline__ void umma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);   // .x = a (low half), .y = b
  return *reinterpret_cast<uint32_t*>(&h);
}

// Tile order: groups of GROUP_M token blocks; inside a group the weight tiles are walked one column
// of the group at a time.  The CTAs that run at the same time then share a few weight tiles and a
// few token blocks (both stay in L2) instead of sweeping the whole weight matrix per token block.
constexpr int GROUP_M = 8;
template <int BN>
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int& m0, int& n0) {
  const int per_group = GROUP_M * tiles_n;
  const int first_m = (tile / per_group) * GROUP_M;
  const int gm = tiles_m - first_m < GROUP_M ? tiles_m - first_m : GROUP_M;
  const int local = tile % per_group;
  m0 = (first_m + local % gm) * BM;
  n0 = (local / gm) * BN;
}

template <int BN, bool PACKED>
__global__ void __launch_bounds__(Shape<BN, PACKED>::N_THREADS, 1)
gemm_tensor_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                   const float* __restrict__ scale, const __grid_constant__ TensorOutputs outs,
                   int32_t* __restrict__ acc_out, int T, int N, int K,
                   int* __restrict__ status) {
  constexpr int STAGES = Shape<BN, PACKED>::STAGES, STAGE_BYTES = Shape<BN, PACKED>::STAGE_BYTES;
  extern __shared__ unsigned char smem_dyn[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t wide_bar[MAX_STAGES];    // PACKED: the stage's token tile has been widened
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t tfull_bar[2];
  __shared__ __align__(8) uint64_t tempty_bar[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;

  unsigned char* tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = (T + BM - 1) / BM, tiles_n = (N + BN - 1) / BN;
  const int n_tiles = tiles_m * tiles_n;
  const int nkb = K / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); mbar_init(&wide_bar[s], WIDEN_THREADS / 32); }
    for (int b = 0; b < 2; ++b) { mbar_init(&tfull_bar[b], 1); mbar_init(&tempty_bar[b], 4); }
    abort_flag_s = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        int m0, n0;
        tile_coords<BN>(tile, tiles_m, tiles_n, m0, n0);
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % STAGES;
          if (!mbar_wait(&empty_bar[s], ((it / STAGES) & 1) ^ 1, abort_flag, status)) { ok = false; break; }
          mbar_expect_tx(&full_bar[s], Shape<BN, PACKED>::TX_BYTES);
          unsigned char* a = tiles + (size_t)s * STAGE_BYTES;
          if constexpr (PACKED) tma_load_2d(a + A_BYTES + Shape<BN, PACKED>::B_BYTES, &tmA, &full_bar[s], kb * (BK / 2), m0);
          else tma_load_2d(a, &tmA, &full_bar[s], kb * BK, m0);
          tma_load_2d(a + A_BYTES, &tmB, &full_bar[s], kb * BK, n0);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      uint32_t it = 0, tl = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tl) {
        const int b = tl & 1;
        if (!mbar_wait(&tempty_bar[b], ((tl >> 1) & 1) ^ 1, abort_flag, status)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)b * BN;
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % STAGES;
          // (the widen warps waited for the stage's copies before they wrote the token tile: one wait covers both)
          if (!mbar_wait(PACKED ? &wide_bar[s] : &full_bar[s], (it / STAGES) & 1, abort_flag, status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(tiles + (size_t)s * STAGE_BYTES);
          const uint64_t adesc = make_desc(a_addr), bdesc = make_desc(a_addr + A_BYTES);
#pragma unroll
          for (int ks = 0; ks < BK / UMMA_K; ++ks)
            umma_i8(d_tmem, adesc + (uint64_t)(ks * UMMA_K / 16), bdesc + (uint64_t)(ks * UMMA_K / 16),
                    Shape<BN, PACKED>::IDESC, (kb | ks) != 0);
          umma_commit(&empty_bar[s]);          // stage reusable once these MMAs have read it
        }
        if (ok) umma_commit(&tfull_bar[b]);    // accumulator complete
      }
    }
  } else if (warp >= THREADS / 32) {
    // ------------------------------ widen (PACKED only) ------------------------------
    // Two threads own token row r of the tile, two 16-byte pieces (32 codes) of its 64 packed bytes each.  The
    // 32-bit word g of a packed row covers elements 8g .. 8g+7, byte b = (q[8g+b] + 8) | (q[8g+b+4] + 8) << 4:
    // `w & 0x0F0F0F0F` is four consecutive codes (plus 8) as bytes, `(w >> 4) & 0x0F0F0F0F` the next four, and a
    // per-byte subtraction of 8 makes them the signed int8 values the MMA reads.  They are written where a
    // 128-byte-swizzled TMA load would have put them: row r at r * 128, its 16-byte chunk c at position c ^ (r & 7).
    if constexpr (PACKED) {
      const int r = ((int)threadIdx.x - THREADS) & (BM - 1);
      const int half = ((int)threadIdx.x - THREADS) >> 7;
      auto widen = [](const uint4& w, uint4& lo, uint4& hi) {
        lo.x = __vsub4(w.x & 0x0F0F0F0Fu, 0x08080808u); lo.y = __vsub4((w.x >> 4) & 0x0F0F0F0Fu, 0x08080808u);
        lo.z = __vsub4(w.y & 0x0F0F0F0Fu, 0x08080808u); lo.w = __vsub4((w.y >> 4) & 0x0F0F0F0Fu, 0x08080808u);
        hi.x = __vsub4(w.z & 0x0F0F0F0Fu, 0x08080808u); hi.y = __vsub4((w.z >> 4) & 0x0F0F0F0Fu, 0x08080808u);
        hi.z = __vsub4(w.w & 0x0F0F0F0Fu, 0x08080808u); hi.w = __vsub4((w.w >> 4) & 0x0F0F0F0Fu, 0x08080808u);
      };
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        for (int kb = 0; kb < nkb; ++kb, ++it) {
          const int s = it % STAGES;
          ok = __all_sync(0xffffffffu, mbar_wait<true>(&full_bar[s], (it / STAGES) & 1, abort_flag, status));
          if (!ok) break;
          unsigned char* stage = tiles + (size_t)s * STAGE_BYTES;
          const unsigned char* pk = stage + A_BYTES + Shape<BN, PACKED>::B_BYTES + r * (BK / 2);
          unsigned char* row = stage + r * BK;
#pragma unroll
          for (int j = 2 * half; j < 2 * half + 2; ++j) {
            // piece order j ^ g(r), g = 0, 2, 3, 1 for (r >> 1) & 3 = 0..3: with it the eight threads of a
            // quarter-warp hit distinct banks both in the loads (row pitch 64 bytes) and in the swizzled stores
            const int jj = j ^ ((0x78 >> (r & 6)) & 3);
            const uint4 w = *reinterpret_cast<const uint4*>(pk + 16 * jj);
            uint4 lo, hi;
            widen(w, lo, hi);
            *reinterpret_cast<uint4*>(row + 16 * ((2 * jj) ^ (r & 7))) = lo;
            *reinterpret_cast<uint4*>(row + 16 * ((2 * jj + 1) ^ (r & 7))) = hi;
          }
          // generic-proxy writes, read next by the tensor cores (async proxy)
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(&wide_bar[s]);
        }
      }
    }
  } else {
    // ------------------------------ epilogue ------------------------------
    const int q = warp & 3;                    // TMEM lane quadrant this warp may access
    uint32_t tl = 0;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tl) {
      const int b = tl & 1;
      int m0, n0;
      tile_coords<BN>(tile, tiles_m, tiles_n, m0, n0);
      const bool got = mbar_wait(&tfull_bar[b], (tl >> 1) & 1, abort_flag, status);
      if (!__all_sync(0xffffffffu, got)) break;      // warp-uniform: tcgen05.ld needs the whole warp
      tc_fence_after();
      const int row = m0 + q * 32 + lane;
      // the weight rows of this tile belong to one output tensor (segments start on tile boundaries)
      int si = 0;
      while (si + 1 < outs.n && n0 >= outs.begin[si + 1]) ++si;
      const int seg_n0 = n0 - outs.begin[si], seg_N = (acc_out != nullptr) ? N : outs.width[si];
      __nv_bfloat16* __restrict__ y = outs.y[si];
      const float f = (acc_out == nullptr && row < T) ? __ldg(scale + row) * __ldg(outs.alpha[si]) : 0.f;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * BN + c * 32), r);
        tmem_ld_wait();
        const int col = seg_n0 + c * 32;
        if (row < T) {
          if (acc_out != nullptr) {
            int32_t* dst = acc_out + (size_t)row * N + col;
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              if (col + i < N) *reinterpret_cast<uint4*>(dst + i) = make_uint4(r[i], r[i + 1], r[i + 2], r[i + 3]);
          } else {
            __nv_bfloat16* dst = y + (size_t)row * seg_N + col;
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              if (col + i < seg_N) {
                uint4 o;
                o.x = pack_bf16((float)(int)r[i + 0] * f, (float)(int)r[i + 1] * f);
                o.y = pack_bf16((float)(int)r[i + 2] * f, (float)(int)r[i + 3] * f);
                o.z = pack_bf16((float)(int)r[i + 4] * f, (float)(int)r[i + 5] * f);
                o.w = pack_bf16((float)(int)r[i + 6] * f, (float)(int)r[i + 7] * f);
                *reinterpret_cast<uint4*>(dst + i) = o;
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty_bar[b]);
    }
  }

  // ------------------------------ teardown ------------------------------
  __syncwarp();
  if (*abort_flag) {
    // give copies that are still in flight time to land before the CTA's shared memory goes away
    const uint64_t t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// ---- host side: tensor maps through the driver entry point (no libcuda link) ----
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// int8 matrix [rows, K] row-major, box = box_rows x 128 bytes, 128-byte swizzle, zero fill.
int make_map(CUtensorMap* map, const void* base, int rows, int K, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return HBL_ERR_CUDA;
  cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)K};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? HBL_OK : HBL_ERR_CUDA;
}

// Packed INT4 codes [rows, K / 2] bytes row-major, box = 128 rows x 64 bytes, no swizzle (the widen warps read it
// row by row), zero fill.
int make_map_packed(CUtensorMap* map, const void* base, int rows, int K) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return HBL_ERR_CUDA;
  cuuint64_t dims[2] = {(cuuint64_t)(K / 2), (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)(K / 2)};
  cuuint32_t box[2] = {(cuuint32_t)(BK / 2), (cuuint32_t)BM};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? HBL_OK : HBL_ERR_CUDA;
}

template <int BN, bool PACKED>
int launch_shape(const void* codes, const float* scale, int T, int K, const int8_t* W_i8, int N, const TensorOutputs& outs,
                 int32_t* acc_out, int n_sm, cudaStream_t s) {
  CUtensorMap tmA, tmB;
  int rc = PACKED ? make_map_packed(&tmA, codes, T, K) : make_map(&tmA, codes, T, K, BM);
  if (rc != HBL_OK) return rc;
  rc = make_map(&tmB, W_i8, N, K, BN);
  if (rc != HBL_OK) return rc;
  auto kern = gemm_tensor_kernel<BN, PACKED>;
  using SH = Shape<BN, PACKED>;
  HBL_ALLOW_DYNAMIC_SMEM(kern, SH::SMEM_BYTES);
  int* status = device_status_word();
  if (status == nullptr) return HBL_ERR_CUDA;
  const int n_tiles = ((T + BM - 1) / BM) * ((N + BN - 1) / BN);
  const int grid = n_tiles < n_sm ? n_tiles : n_sm;
  profile_before(KERNEL_CONTRACT, s);
  kern<<<grid, SH::N_THREADS, SH::SMEM_BYTES, s>>>(tmA, tmB, scale, outs, acc_out, T, N, K, status);
  profile_after(KERNEL_CONTRACT, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

}  // namespace

int launch_gemm_tensor_multi(const void* codes, bool codes_packed, const float* scale, int T, int K, const int8_t* W_i8,
                             const TensorOutputs& outs, int32_t* acc_out, cudaStream_t s) {
  if (T <= 0) return HBL_OK;
  if (outs.n < 1 || outs.n > kMaxTensorOutputs) return HBL_ERR_SHAPE;
  int N = 0;
  for (int i = 0; i < outs.n; ++i) {
    if (outs.begin[i] != N || outs.width[i] <= 0) return HBL_ERR_SHAPE;
    if (i + 1 < outs.n && outs.width[i] % 256 != 0) return HBL_ERR_SHAPE;    // a tile never straddles two outputs
    N += outs.width[i];
  }
  const int n_sm = sm_count();
  // The narrow tile only pays on very small grids, where even twice as many tiles leave half of the SMs
  // idle (measured: 2048 x 2048 at 256 tokens 14.3 -> 12.8 us).  It costs about 1.5x per weight row (a
  // 128 x 128 x 32 MMA reads as much of the token block from shared memory as a 128 x 256 x 32 one), and at
  // larger sizes small-batch contractions are bound by L2 traffic, which narrower tiles increase
  // (8192 -> 2048 at 1024 tokens: 37.6 -> 39.2 us; a 7B block at 4096 tokens: 0.96 -> 1.13 ms).
  const long t128 = (long)((T + BM - 1) / BM) * ((N + 127) / 128);
  const bool narrow = N > 128 && 2 * t128 <= n_sm;
  if (codes_packed) {
    if (narrow) return launch_shape<128, true>(codes, scale, T, K, W_i8, N, outs, acc_out, n_sm, s);
    return launch_shape<256, true>(codes, scale, T, K, W_i8, N, outs, acc_out, n_sm, s);
  }
  if (narrow) return launch_shape<128, false>(codes, scale, T, K, W_i8, N, outs, acc_out, n_sm, s);
  return launch_shape<256, false>(codes, scale, T, K, W_i8, N, outs, acc_out, n_sm, s);
}

int launch_gemm_tensor(const void* codes, bool codes_packed, const float* scale, int T, int K, const int8_t* W_i8, int N,
                       const float* alpha, __nv_bfloat16* y, int32_t* acc_out, cudaStream_t s) {
  TensorOutputs outs = {};
  outs.n = 1; outs.begin[0] = 0; outs.width[0] = N; outs.y[0] = y; outs.alpha[0] = alpha;
  return launch_gemm_tensor_multi(codes, codes_packed, scale, T, K, W_i8, outs, acc_out, s);
}

}  // namespace hbl
