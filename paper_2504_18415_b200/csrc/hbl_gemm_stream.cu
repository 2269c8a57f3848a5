// Small-batch contraction of H-BitLinear (Eq. 7) for T <= 128 tokens, bound by the
// stream of 2-bit packed weights out of HBM.
//
// The roles are swapped with respect to the large-batch kernel: 128 weight rows
// are the M side of tcgen05.mma kind::i8 and the (padded) tokens the N side, so a
// step of 128 x T x 32 costs a few cycles of the tensor core and the int32 sums of
// a whole K range stay in tensor memory -- no partial sums ever cross shared
// memory.  The A operand is read from tensor memory too: unpack warps expand the
// 2-bit weights to unsigned bytes in registers (one shift-and-mask per four
// weights) and write them with tcgen05.st, so the expanded weights never touch
// shared memory either.  What crosses shared memory is the packed stream (once in
// by bulk copy, once out by 128-bit loads) and the tokens' codes (TMA).
//
//   warp 0        weight producer: one bulk copy per unit (KBP packed tiles of 4 KiB, contiguous),
//                 the first ring-full issued before anything else in the kernel
//   warp 2        codes producer: TMA loads of the unit's codes [T_pad x 128] per column block,
//                 a ring of their own
//   warp 1 (, 3)  warp 1 allocates tensor memory; an issuer warp stays converged and one elected
//                 lane issues the MMAs; up to 32 token columns warps 1 and 3 issue half a unit each
//   warps 4..11   unpack: two groups of four warps (one per TMEM lane quadrant) take alternate
//                 units and hand the weight stage back as soon as its words are in registers
//   warps 12..15  epilogue: read the accumulators (two D buffers alternate), divide by 64 and subtract
//                 the code sum (weights are fed as 64 (w + 1)), rescale, store bf16
//
// Work is dealt stream-K style: all (row block, column block) pairs in row-major
// order, cut into equal contiguous ranges, one per CTA, so every SM streams the
// same number of bytes.  A row block whose range is cut belongs to the CTA that
// holds its first column block; the other CTAs write their partial sums to a slot
// of their own in `part`, raise a flag, and the owner adds them when its own range
// is done.  A CTA publishes before it ever waits, so the waits cannot cycle; every
// wait is bounded and reports HBL_ERR_TIMEOUT.
#include <cuda.h>

#include "hbl_pipeline.cuh"

namespace hbl {
namespace {

using namespace pipe;

constexpr int THREADS = 512;
constexpr int MAX_SW = 16;             // weight stages in shared memory
constexpr int MAX_SC = 8;              // codes stages
constexpr int MAX_NA = 12;             // A buffers in tensor memory
// Tensor memory: two D buffers of D_COLS columns each, then the A buffers.
constexpr int SMEM_RING_BYTES = 192 * 1024;
constexpr int TMEM_COLS = 512;
constexpr int TILE_BYTES = 4096;       // 128 rows x 128 columns x 2 bits
constexpr int MAX_GRID = 160;
// The unpack warps leave each 2-bit field u = w + 1 in the top two bits of its byte (a left shift
// and a mask; no right shifts), so the MMA sees 64 u and every accumulator is an exact multiple of 64.
constexpr int WEIGHT_SHIFT = 6;

constexpr int MAX_JOBS = 8;            // weight tensors contracted by one launch (a decoder block has seven)
constexpr int MAX_MAPS = 4;            // distinct quantized inputs they read (a decoder block has four)

// One weight tensor and where its result goes.  Units (KBP column blocks of one row block) are
// numbered across all jobs of a launch: this job's are [u_begin, u_begin + n_rb * n_kb).
struct Job {
  const unsigned char* Wp; const float* scale; const int32_t* codesum; const float* alpha;
  __nv_bfloat16* y; int32_t* acc_out;
  int N, n_kb, map;
  uint32_t u_begin;
};
struct Params {
  Job jobs[MAX_JOBS];
  int n_jobs;
  uint32_t U;         // units of all jobs (U * grid fits 32 bits: checked on the host)
  int32_t* part;      // [grid][t_pad][128] partial sums of row blocks this CTA does not own
  int* flags;         // [grid], zero on entry
  int* status;
  int T;
  int release_early;  // release the programmatic dependents once the kernel before this one is known to be complete
  // Back-to-back mode: the quantizer of this call ran beside the previous contraction and completes only when that
  // one does.  Its thread blocks count themselves in per input (ready[m], counters the library owns) once their
  // codes are written, and the codes producer waits for those counts instead of the quantizer's completion, so the
  // MMAs start while the previous contraction still drains; the epilogue keeps waiting for completion.
  const unsigned* ready;          // nullptr: wait for the kernel before this one as a whole
  unsigned ready_target[MAX_MAPS];
  unsigned* done;                 // non-null: thread blocks of this launch that are through; the last one clears ready[] and done
  int done_early;                 // count in as soon as the codes producer has read the counters for the last time
                                  // (single launch per call); else at the end of the kernel (last of several passes)
};
struct CodeMaps { CUtensorMap m[MAX_MAPS]; };   // codes [T, K] of each input, box 128 x T_pad, 128-byte swizzle

// Instruction descriptor: D s32 (2 << 4), A unsigned 8-bit (0 << 7), B signed 8-bit (1 << 10),
// both K-major, N >> 3 at bit 17, M >> 4 at bit 24.
__device__ __forceinline__ uint32_t make_idesc(int n_tok) {
  return (2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(n_tok >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
// Shared-memory matrix descriptor, K-major, 128-byte swizzle, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
  return (uint64_t)((saddr >> 4) & 0x3FFF) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void umma_i8_tmem_a(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], %2, %3, p;\n}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Acquire load at GPU scope: what the writer stored before its release of the flag is visible after it.
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Waits (bounded) until a counter that another kernel's thread blocks raise has reached `target`.  That kernel was
// launched before this one and waits for nothing this one does.
__device__ __forceinline__ bool wait_count(const unsigned* counter, unsigned target, volatile int* abort_flag, int* status) {
  const uint64_t t0 = global_ns();
  for (uint32_t polls = 0;; ++polls) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= target) break;
    if (*abort_flag) return false;
    if ((polls & 63u) == 63u && global_ns() - t0 > kWaitLimitNs) {
      report_device_error(status, HBL_ERR_TIMEOUT);
      *abort_flag = 1;
      return false;
    }
    __nanosleep(100);
  }
  asm volatile("fence.proxy.async.global;" ::: "memory");   // the bulk tensor copies that follow read what the counter covers
  return true;
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// One lane of a converged warp.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n .reg .pred p;\n elect.sync _|p, 0xffffffff;\n selp.u32 %0, 1, 0, p;\n}" : "=r"(pred));
  return pred != 0;
}
// A whole warp waits on a barrier and stays converged.  (Measured: a wait that is satisfied at once
// costs the warp about 95 cycles this way, about 150 when one lane polls and hands the outcome
// round, and the whole kernel ran slower with single-lane polling -- so every lane polls, and the
// serial loops below are arranged to need as few waits per unit as possible.)
template <bool POLITE>
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status) {
  return __all_sync(0xffffffffu, mbar_wait<POLITE>(bar, parity, abort_flag, status));
}
template <bool POLITE>
__device__ __forceinline__ bool warp_wait2(uint64_t* bar0, uint32_t parity0, uint64_t* bar1, uint32_t parity1,
                                           volatile int* abort_flag, int* status) {
  return __all_sync(0xffffffffu, mbar_wait<POLITE>(bar0, parity0, abort_flag, status) &&
                                     mbar_wait<POLITE>(bar1, parity1, abort_flag, status));
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}

// One contiguous piece of a CTA's range: units [ka, ke) of row block rb of one job.
struct Segment { int job, rb, ka, ke; uint32_t rb_end; /* global index one past the row block's last unit */ };
struct Range {
  const Params& p;
  uint32_t u1, pos;   // 32-bit on purpose: every role walks its range with these divisions
  __device__ Range(const Params& p_, uint32_t u0_, uint32_t u1_) : p(p_), u1(u1_), pos(u0_) {}
  __device__ bool next(Segment& s) {
    if (pos >= u1) return false;
    int j = 0;
    while (j + 1 < p.n_jobs && pos >= p.jobs[j + 1].u_begin) ++j;
    const uint32_t local = pos - p.jobs[j].u_begin;
    const uint32_t n_kb = (uint32_t)p.jobs[j].n_kb;
    s.job = j;
    s.rb = (int)(local / n_kb);
    s.ka = (int)(local % n_kb);
    s.rb_end = p.jobs[j].u_begin + (uint32_t)(s.rb + 1) * n_kb;
    s.ke = (int)((u1 < s.rb_end ? u1 : s.rb_end) - (s.rb_end - n_kb));
    pos = s.rb_end - n_kb + s.ke;
    return true;
  }
};

// A unit of work is KBP consecutive 128-column blocks of one row block.  Its packed weights are one
// contiguous run of KBP x 4 KiB (one bulk copy: copies of 16 KiB or more are what keeps HBM busy),
// its codes KBP boxes of [T_PAD x 128].  The two travel in rings of their own: a weight stage is
// handed back as soon as the unpack warps hold its words in registers, a codes stage when the MMAs
// that read it have completed.
template <int T_PAD, int KBP>
struct Geo {
  static constexpr int W_BYTES = KBP * TILE_BYTES;
  static constexpr int C_BYTES = KBP * T_PAD * 128;
  // The codes come from L2 but queue behind the weight traffic, so they need the same lookahead
  // in units as the weights: the ring bytes are split into equally many stages of each.
  static constexpr int SC_RAW = SMEM_RING_BYTES / (C_BYTES + W_BYTES);
  static constexpr int SC_CAP = SC_RAW > MAX_SC ? MAX_SC : SC_RAW;
  static constexpr int SC = SC_CAP > 1 ? (SC_CAP & ~1) : SC_CAP;   // even: a stage stays with one issuer
  static constexpr int SW_RAW = (SMEM_RING_BYTES - SC * C_BYTES) / W_BYTES;
  static constexpr int SW_CAP = SW_RAW > MAX_SW ? MAX_SW : SW_RAW;
  static constexpr int SW = SW_CAP & ~1;                          // even: a stage stays with one unpack group
  // One thread issues an MMA every ~25 cycles, a unit of four tiles takes sixteen plus the waits and
  // commits around them: more than the ~700 cycles in which HBM delivers the unit.  Up to 32 token
  // columns two warps issue, each one half of every unit's MMAs into an accumulator of its own (the
  // epilogue adds the two).  Both walk the units in the same order, so every barrier still sees its
  // phases complete one at a time (issuers on alternate units would let one run two phases ahead of
  // the other, which a parity wait cannot tell from "not yet").  Beyond 32 columns tensor memory has
  // no room for the second accumulator set and the path is no longer bound by the weight stream.
  static constexpr int ISSUERS = T_PAD <= 32 ? 2 : 1;
  static constexpr int D_COLS = T_PAD < 64 ? 64 : T_PAD;          // columns of one accumulator buffer (all issuers)
  static constexpr int D_ISSUER_COLS = D_COLS / ISSUERS;
  static constexpr int A_COL0 = 2 * D_COLS;
  static constexpr int NA_RAW = (TMEM_COLS - A_COL0) / (32 * KBP);
  static constexpr int NA = NA_RAW > MAX_NA ? MAX_NA : NA_RAW;
  static constexpr int W_OFF = SC * C_BYTES;                      // codes ring first (1024-byte aligned boxes)
  static constexpr size_t SMEM = (size_t)SC * C_BYTES + (size_t)SW * W_BYTES + 1024;
};

template <int T_PAD, int KBP>
__global__ void __launch_bounds__(THREADS, 1)
gemm_stream_kernel(const __grid_constant__ CodeMaps maps, const __grid_constant__ Params p) {
  using GEO = Geo<T_PAD, KBP>;
  constexpr int SW = GEO::SW, SC = GEO::SC, NA = GEO::NA, D_COLS = GEO::D_COLS, A_COL0 = GEO::A_COL0;
  constexpr int W_BYTES = GEO::W_BYTES, C_BYTES = GEO::C_BYTES, ISSUERS = GEO::ISSUERS;
  extern __shared__ unsigned char smem_dyn[];
  __shared__ __align__(8) uint64_t w_full[MAX_SW], w_empty[MAX_SW], c_full[MAX_SC], c_empty[MAX_SC], a_full[MAX_NA],
      a_empty[MAX_NA], d_full[2], d_empty[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;
  unsigned char* c_ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  unsigned char* w_ring = c_ring + GEO::W_OFF;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t U = p.U;
  const int G = gridDim.x, c = blockIdx.x;
  const uint32_t u0 = U * (uint32_t)c / (uint32_t)G, u1 = U * (uint32_t)(c + 1) / (uint32_t)G;

  if (tid == 0) {
    for (int s = 0; s < SW; ++s) { mbar_init(&w_full[s], 1); mbar_init(&w_empty[s], 4); }
    for (int s = 0; s < SC; ++s) { mbar_init(&c_full[s], 1); mbar_init(&c_empty[s], ISSUERS); }
    for (int a = 0; a < NA; ++a) { mbar_init(&a_full[a], 4); mbar_init(&a_empty[a], ISSUERS); }
    for (int b = 0; b < 2; ++b) { mbar_init(&d_full[b], ISSUERS); mbar_init(&d_empty[b], 4); }
    abort_flag_s = 0;
    mbar_fence_init();
  }
  // The packed weights depend on no earlier kernel: the first ring-full of copies leaves before
  // the CTA has even allocated its tensor memory, and (programmatic dependent launch) while the
  // kernel that quantizes the activations may still be running.  Lane l of warp 0 issues stage l's.
  const uint32_t primed = (u1 - u0) < (uint32_t)SW ? (u1 - u0) : (uint32_t)SW;
  if (warp == 0) {
    __syncwarp();
    if ((uint32_t)lane < primed) {
      const uint32_t u = u0 + (uint32_t)lane;
      int j = 0;
      while (j + 1 < p.n_jobs && u >= p.jobs[j + 1].u_begin) ++j;
      const Job& job = p.jobs[j];
      mbar_expect_tx(&w_full[lane], W_BYTES);
      // units of a job lie in memory in the order they are numbered
      bulk_load(w_ring + (size_t)lane * W_BYTES, job.Wp + (size_t)(u - job.u_begin) * W_BYTES, W_BYTES, &w_full[lane]);
    }
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
    // ------------------------------ weight producer ------------------------------
    if (lane == 0) {
      Range range(p, u0, u1);
      Segment sg;
      uint32_t i = 0;
      bool ok = true;
      while (ok && range.next(sg)) {
        const Job& job = p.jobs[sg.job];
        for (int kb = sg.ka; kb < sg.ke; ++kb, ++i) {
          if (i < primed) continue;
          const int s = i % SW;
          if (!mbar_wait<true>(&w_empty[s], ((i / SW) & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
          mbar_expect_tx(&w_full[s], W_BYTES);
          bulk_load(w_ring + (size_t)s * W_BYTES, job.Wp + ((size_t)sg.rb * job.n_kb + kb) * W_BYTES, W_BYTES, &w_full[s]);
        }
      }
    }
  } else if (warp == 2) {
    // ------------------------------ codes producer ------------------------------
    if (lane == 0) {
      uint32_t complete = 0;                                   // inputs whose codes are known to be written
      if (p.ready == nullptr) {
        grid_dependency_wait();                                // the codes come from the previous kernel
        complete = ~0u;
      }
      Range range(p, u0, u1);
      Segment sg;
      uint32_t i = 0;
      bool ok = true;
      while (ok && range.next(sg)) {
        const int in = p.jobs[sg.job].map;
        if (!((complete >> in) & 1u)) {
          if (!wait_count(p.ready + in, p.ready_target[in], abort_flag, p.status)) break;
          complete |= 1u << in;
        }
        const CUtensorMap* tm_codes = &maps.m[in];
        for (int kb = sg.ka; kb < sg.ke; ++kb, ++i) {
          const int s = i % SC;
          if (i >= (uint32_t)SC && !mbar_wait<true>(&c_empty[s], ((i / SC) & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
          mbar_expect_tx(&c_full[s], C_BYTES);
#pragma unroll
          for (int j = 0; j < KBP; ++j)
            tma_load_2d(c_ring + (size_t)s * C_BYTES + j * (T_PAD * 128), tm_codes, &c_full[s], (kb * KBP + j) * 128, 0);
        }
      }
      // This thread is the only one of the CTA that reads the quantizer's counters, and it is through with them.
      // Once the producers of all CTAs of the launch have come by here, the last one puts the counters back to
      // zero for the next call that uses this half (here rather than at the end of the kernel: the answer of the
      // atomic is a trip to L2, which the CTA's last stores should not have to wait for).  Only where the call is
      // this one launch: with several passes a CTA of an earlier pass may not have read all its counters yet.
      if (p.done != nullptr && p.done_early && atomicAdd(p.done, 1u) == gridDim.x - 1) {
        unsigned* ready = const_cast<unsigned*>(p.ready);
        for (int m = 0; m < MAX_MAPS; ++m) atomicExch(ready + m, 0u);
        atomicExch(p.done, 0u);
      }
    }
  } else if (warp == 1 || (ISSUERS == 2 && warp == 3)) {
    // ------------------------------ MMA issuer(s) ------------------------------
    // The whole warp walks the loop and one elected lane issues: in warp-uniform code the operands
    // of tcgen05.mma (descriptors, tensor-memory addresses) live in uniform registers, and the
    // instructions issue several times faster than from inside a single-lane branch.
    const int g = warp >> 1;                                   // issuer 0 or 1
    constexpr int MMAS = 4 * KBP / ISSUERS;                    // this issuer's share of a unit's MMAs
    const uint32_t idesc = make_idesc(T_PAD);
    Range range(p, u0, u1);
    Segment sg;
    uint32_t i = 0, seg = 0;
    bool ok = true;
    while (ok && range.next(sg)) {
      const int b = seg & 1;
      ok = warp_wait<false>(&d_empty[b], ((seg >> 1) & 1) ^ 1, abort_flag, p.status);
      if (!ok) break;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(b * D_COLS + g * GEO::D_ISSUER_COLS);
      uint32_t accumulate = 0;                                 // this issuer's first MMA of the segment overwrites
      for (int kb = sg.ka; kb < sg.ke; ++kb, ++i) {
        const int s = i % SC, a = i % NA;
        // The unpack warps waited for the unit's codes before they filled the A buffer, so this one
        // wait covers both operands.
        ok = warp_wait<false>(&a_full[a], (i / NA) & 1, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t codes_sm = smem_u32(c_ring + (size_t)s * C_BYTES);
        const uint32_t a_tmem = tmem_base + A_COL0 + (uint32_t)(32 * KBP) * a;
        if (elect_one()) {
#pragma unroll
          for (int q = 0; q < MMAS; ++q) {
            const int m = g * MMAS + q, j = m >> 2, ks = m & 3;   // MMA m of the unit: tile j, K step ks
            const uint64_t bdesc = make_desc(codes_sm + j * (T_PAD * 128));
            umma_i8_tmem_a(d_tmem, a_tmem + 32u * j + 8u * ks, bdesc + (uint64_t)(2 * ks), idesc,
                           accumulate | (uint32_t)(q > 0));
          }
          umma_commit(&c_empty[s]);          // the stage's codes have been read
          umma_commit(&a_empty[a]);          // and so has the A buffer
        }
        accumulate = 1;
        __syncwarp();
      }
      // elect.sync names the same lane for the same mask every time, so this commit tracks the MMAs above
      if (ok && elect_one()) umma_commit(&d_full[b]);
      __syncwarp();
      ++seg;
    }
  } else if (warp >= 4 && warp < 12) {
    // ------------------------------ unpack ------------------------------
    // Two groups of four warps (one per TMEM lane quadrant) take alternate units, so one group's
    // waits and tensor-memory stores overlap the other's arithmetic.  A warp first pulls all of the
    // unit's words for its 32 rows into registers, then expands them tile by tile.
    const int group = (warp - 4) >> 2, quad = warp & 3;
    const int row = quad * 32 + lane;
    Range range(p, u0, u1);
    Segment sg;
    uint32_t i = 0;
    bool ok = true;
    while (ok && range.next(sg)) {
      for (int kb = sg.ka; kb < sg.ke; ++kb, ++i) {
        if ((int)(i & 1) != group) continue;
        const int s = i % SW, sc = i % SC, a = i % NA;
        ok = warp_wait<true>(&w_full[s], (i / SW) & 1, abort_flag, p.status);
        if (!ok) break;
        const unsigned char* st = w_ring + (size_t)s * W_BYTES + row * 16;
        uint4 w4[KBP][2];
#pragma unroll
        for (int j = 0; j < KBP; ++j) {
          w4[j][0] = *reinterpret_cast<const uint4*>(st + j * TILE_BYTES);
          w4[j][1] = *reinterpret_cast<const uint4*>(st + j * TILE_BYTES + 2048);
        }
        // the codes must have landed before the MMA warp is told that the unit is ready
        ok = warp_wait2<true>(&c_full[sc], (i / SC) & 1, &a_empty[a], ((i / NA) & 1) ^ 1, abort_flag, p.status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = tmem_base + A_COL0 + (uint32_t)(32 * KBP) * a + ((uint32_t)(quad * 32) << 16);
#pragma unroll
        for (int j = 0; j < KBP; ++j) {
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const uint32_t w[4] = {w4[j][h].x, w4[j][h].y, w4[j][h].z, w4[j][h].w};
            uint32_t r[16];
#pragma unroll
            for (int kq = 0; kq < 4; ++kq)
#pragma unroll
              for (int q = 0; q < 4; ++q) r[kq * 4 + q] = (w[kq] << (6 - 2 * q)) & 0xC0C0C0C0u;   // k = 64 h + 16 kq + 4 q + byte
            tmem_st16(a_addr + 32u * j + 16u * h, r);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&w_empty[s]);               // the words are in registers: the stage can be refilled
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&a_full[a]);
      }
    }
  } else if (warp >= 12) {
    // ------------------------------ epilogue ------------------------------
    // Accumulators are handled 16 token columns at a time, so nothing here needs more than a few
    // dozen registers whatever T_PAD is.
    grid_dependency_wait();                                  // scales, code sums and cleared flags come from the previous kernel
    // Back-to-back mode: only now may the next call's quantizer start (it runs beside this kernel and may be followed
    // by another contraction; the wait above has seen everything before this kernel complete, so at most two calls
    // are ever in flight and the half of the scratch the next quantizer writes is no longer read by anyone).
    if (p.release_early && warp == 12 && lane == 0) grid_launch_dependents();
    const int quad = warp & 3;
    const int row_in_block = quad * 32 + lane;
    const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16);
    // The job's fields are copied to registers once per segment (the job table sits in parameter
    // space; indexing it dynamically inside the store loop would re-read it every time).
    struct Out { const float* scale; const int32_t* codesum; __nv_bfloat16* y; int32_t* acc_out; float al; int N; };
    auto job_out = [&](int job_idx) {
      const Job& job = p.jobs[job_idx];
      Out o;
      o.scale = job.scale; o.codesum = job.codesum; o.y = job.y; o.acc_out = job.acc_out; o.N = job.N;
      o.al = (job.acc_out == nullptr) ? __ldg(job.alpha) : 0.f;
      return o;
    };
    // Lane t (mod 16) fetches the code sum and the scale of token 16 j + t; finish_chunk hands them
    // round by shuffle.  Fetched ahead of the wait for the accumulators, so the loads overlap it.
    struct Tok { int cs; float s; };
    auto fetch_tok = [&](const Out& o, int j) {
      const int my_tok = j * 16 + (lane & 15);
      Tok t;
      t.cs = my_tok < p.T ? __ldg(o.codesum + my_tok) : 0;
      t.s = (my_tok < p.T && o.acc_out == nullptr) ? __ldg(o.scale + my_tok) : 0.f;
      return t;
    };
    auto finish_chunk = [&](const Out& o, int rb, int j, const Tok& mine, const int (&v)[16]) {
      const int row = rb * 128 + row_in_block;
      const float my_f = mine.s * o.al;
#pragma unroll
      for (int t = 0; t < 16; ++t) {
        const int tok = j * 16 + t;
        const int cs = __shfl_sync(0xffffffffu, mine.cs, t);
        const float f = __shfl_sync(0xffffffffu, my_f, t);
        if (tok < p.T && row < o.N) {
          const int a = (v[t] >> WEIGHT_SHIFT) - cs;
          if (o.acc_out != nullptr) o.acc_out[(size_t)tok * o.N + row] = a;
          else o.y[(size_t)tok * o.N + row] = __float2bfloat16_rn((float)a * f);
        }
      }
    };
    auto load_chunk = [&](int b, int j, int (&v)[16]) {
      uint32_t r[16];
      tmem_ld16(lane_base + (uint32_t)(b * D_COLS + j * 16), r);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
      for (int t = 0; t < 16; ++t) v[t] = (int)r[t];
      if (ISSUERS == 2) {
        tmem_ld16(lane_base + (uint32_t)(b * D_COLS + GEO::D_ISSUER_COLS + j * 16), r);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int t = 0; t < 16; ++t) v[t] += (int)r[t];
      }
    };
    const int n_chunks = (p.T + 15) / 16;
    Range range(p, u0, u1);
    Segment sg;
    uint32_t seg = 0;
    bool ok = true;
    // A row block this CTA owns but does not complete is its last segment: its sums stay in their
    // D buffer until the other CTAs' parts have been added.
    int own_b = -1, own_rb = 0, n_follow = 0;
    Out own_o = {};
    Tok own_tok0 = {0, 0.f};
    while (range.next(sg)) {
      const int b = seg & 1;
      const bool whole = sg.ka == 0 && sg.ke == p.jobs[sg.job].n_kb;
      const bool own_partial = sg.ka == 0 && !whole;
      Out o;
      Tok tok0 = {0, 0.f};
      if (whole || own_partial) { o = job_out(sg.job); tok0 = fetch_tok(o, 0); }
      if (own_partial) {
        // Everything that needs neither the accumulators nor the other CTAs' parts happens before the
        // wait: this segment is the CTA's last, so what follows it is the tail of the whole kernel.
        own_o = o; own_tok0 = tok0;
        while (c + 1 + n_follow < G && U * (uint32_t)(c + 1 + n_follow) / (uint32_t)G < sg.rb_end) ++n_follow;
      }
      ok = ok && warp_wait<true>(&d_full[b], (seg >> 1) & 1, abort_flag, p.status);
      ++seg;
      if (own_partial) {
        if (ok) { own_b = b; own_rb = sg.rb; }
        continue;
      }
      if (ok) {
        tc_fence_after();
#pragma unroll 1
        for (int j = 0; j < T_PAD / 16; ++j) {
          if (j >= n_chunks) break;                           // padded token columns are never read
          int v[16];
          load_chunk(b, j, v);
          if (whole) {
            finish_chunk(o, sg.rb, j, j == 0 ? tok0 : fetch_tok(o, j), v);
          } else {
            // not the owner: publish the partial sums ([token][128 rows], coalesced)
#pragma unroll
            for (int t = 0; t < 16; ++t) __stcg(p.part + ((size_t)c * T_PAD + j * 16 + t) * 128 + row_in_block, v[t]);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&d_empty[b]);
      }
      if (!whole) {
        if (ok) __threadfence();
        named_barrier(3, 128);                                // all four epilogue warps have written their rows
        if (ok && warp == 12 && lane == 0) atomicExch(p.flags + c, 1);
      }
    }
    if (own_b >= 0 && ok) {
      // the row block continues in the next CTAs: collect their parts (each was published before its CTA waits for anything)
      const Out& o = own_o;
      const Tok& tok0 = own_tok0;
      {
        int ready = 1;                                        // lane l polls the flags of followers l, l+32, ...
        for (int f = lane; f < n_follow && ready; f += 32) {
          const int* flag = p.flags + c + 1 + f;
          if (ld_acquire(flag)) continue;                     // the usual case: published long ago
          const uint64_t t0 = global_ns();
          while (!ld_acquire(flag)) {
            if (*abort_flag) { ready = 0; break; }
            if (global_ns() - t0 > 2000000000ull) {
              report_device_error(p.status, HBL_ERR_TIMEOUT);
              *abort_flag = 1;
              ready = 0;
              break;
            }
            __nanosleep(64);
          }
        }
        ok = __all_sync(0xffffffffu, ready);
      }
      if (ok) {
        tc_fence_after();
#pragma unroll 1
        for (int j = 0; j < T_PAD / 16; ++j) {
          if (j >= n_chunks) break;
          int v[16];
          load_chunk(own_b, j, v);
          for (int f0 = 0; f0 < n_follow; f0 += 4) {          // independent loads, four followers in flight
            int tmp[4][16];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const int f = f0 + q < n_follow ? f0 + q : n_follow - 1;
#pragma unroll
              for (int t = 0; t < 16; ++t)
                tmp[q][t] = __ldcg(p.part + ((size_t)(c + 1 + f) * T_PAD + j * 16 + t) * 128 + row_in_block);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
              if (f0 + q < n_follow) {
#pragma unroll
                for (int t = 0; t < 16; ++t) v[t] += tmp[q][t];
              }
          }
          finish_chunk(o, own_rb, j, j == 0 ? tok0 : fetch_tok(o, j), v);
        }
        tc_fence_before();
      }
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
  if (p.done != nullptr && !p.done_early && tid == 0) {
    // last of several passes: every epilogue of this launch has waited for the passes before it to complete, so
    // when all CTAs have come by here nobody reads the quantizer's counters any more
    if (atomicAdd(p.done, 1u) == gridDim.x - 1) {
      unsigned* ready = const_cast<unsigned*>(p.ready);
      for (int m = 0; m < MAX_MAPS; ++m) atomicExch(ready + m, 0u);
      atomicExch(p.done, 0u);
    }
  }
}

// ---- host side ----
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

int pad_tokens(int T) { return T <= 16 ? 16 : (T <= 32 ? 32 : (T <= 64 ? 64 : 128)); }

template <int T_PAD, int KBP>
int launch_variant(const CodeMaps& maps, const Params& p, int grid, cudaStream_t s) {
  using GEO = Geo<T_PAD, KBP>;
  constexpr size_t smem = GEO::SMEM;
  auto kern = gemm_stream_kernel<T_PAD, KBP>;
  HBL_ALLOW_DYNAMIC_SMEM(kern, smem);
  // Programmatic dependent launch: if the previous operation on the stream is a kernel that signals
  // griddepcontrol.launch_dependents (the activation kernels do), this kernel may start while it runs.
  profile_before(KERNEL_CONTRACT, s);
  launch_mode().releases_early = p.release_early != 0;
  const cudaError_t launched = launch_dependent(kern, dim3((unsigned)grid), dim3(THREADS), smem, s, maps, p);
  launch_mode().releases_early = false;
  HBL_CUDA_OK(launched);
  profile_after(KERNEL_CONTRACT, s);
  note_launch();
  HBL_CUDA_OK(cudaGetLastError());
  return HBL_OK;
}

template <int T_PAD>
int launch_kbp(int kbp, const CodeMaps& maps, const Params& p, int grid, cudaStream_t s) {
  if (kbp == 4) return launch_variant<T_PAD, 4>(maps, p, grid, s);
  if (kbp == 2) return launch_variant<T_PAD, 2>(maps, p, grid, s);
  return launch_variant<T_PAD, 1>(maps, p, grid, s);
}

}  // namespace

// Scratch of the streaming contraction: `part` slots (contents irrelevant on entry) and flags (zero on
// entry; one set per pass of 128 tokens).
constexpr int kMaxPasses = 4;
size_t gemm_stream_acc_words(int T, int N) {
  (void)N;
  return (size_t)MAX_GRID * 128 * pad_tokens(T < 1 ? 1 : (T > 128 ? 128 : T));
}
size_t gemm_stream_counter_words(int N) { (void)N; return (size_t)MAX_GRID * kMaxPasses; }
int gemm_stream_max_tokens() { return 128 * kMaxPasses; }

// Several weight tensors (each reading one of up to four quantized inputs) in one launch, T <= 128.
static int launch_gemm_stream_pass(const StreamInput* inputs, int n_inputs, const StreamJob* jobs, int n_jobs, int T,
                             int32_t* part, int* flags, cudaStream_t s, int early_release_reserve,
                             const StreamReady* ready, bool last_pass, bool single_pass) {
  if (T <= 0 || n_jobs <= 0) return HBL_OK;
  if (T > 128) return HBL_ERR_TOO_LARGE;
  if (n_jobs > MAX_JOBS || n_inputs > MAX_MAPS || n_inputs <= 0) return HBL_ERR_SHAPE;
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return HBL_ERR_CUDA;
  const int t_pad = pad_tokens(T);
  CodeMaps maps;
  for (int m = 0; m < MAX_MAPS; ++m) {
    if (m >= n_inputs) { maps.m[m] = maps.m[0]; continue; }   // unused slots: any valid map
    // codes [T, K] int8 row-major; box = 128 bytes of K x t_pad tokens (rows beyond T read as zero), 128-byte swizzle
    const StreamInput& in = inputs[m];
    cuuint64_t dims[2] = {(cuuint64_t)in.K, (cuuint64_t)T};
    cuuint64_t strides[1] = {(cuuint64_t)in.K};
    cuuint32_t box[2] = {128u, (cuuint32_t)t_pad};
    cuuint32_t estr[2] = {1, 1};
    if (fn(&maps.m[m], CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(in.codes), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return HBL_ERR_CUDA;
  }
  int n_sm = sm_count();
  if (n_sm > MAX_GRID) n_sm = MAX_GRID;
  const int n_sm_all = n_sm;
  // (a contraction that releases its dependents early leaves SMs free for them: at most 20, beyond which the
  //  missing thread blocks cost more than the next call's quantizer gains by starting early)
  if (early_release_reserve > 0) n_sm -= early_release_reserve < 20 ? early_release_reserve : 20;
  // Column blocks per unit: as wide as every K allows while every CTA still gets a few units.
  long blocks = 0;
  for (int j = 0; j < n_jobs; ++j) blocks += (long)((jobs[j].N + 127) / 128) * (inputs[jobs[j].input].K / 128);
  int kbp = t_pad > 64 ? 2 : 4;            // 128 token columns: the codes of a unit fill the stage, keep units at two blocks
  for (;;) {
    bool fits = blocks / kbp >= 4L * n_sm;
    for (int m = 0; m < n_inputs; ++m) fits = fits && (inputs[m].K / 128) % kbp == 0;
    if (fits || kbp == 1) break;
    kbp >>= 1;
  }
  Params p;
  p.n_jobs = n_jobs;
  long u = 0;
  for (int j = 0; j < n_jobs; ++j) {
    const StreamInput& in = inputs[jobs[j].input];
    Job& jb = p.jobs[j];
    jb.Wp = static_cast<const unsigned char*>(jobs[j].W_packed);
    jb.scale = in.scale; jb.codesum = in.codesum; jb.alpha = jobs[j].alpha;
    jb.y = jobs[j].y; jb.acc_out = jobs[j].acc_out;
    jb.N = jobs[j].N; jb.n_kb = in.K / (128 * kbp); jb.map = jobs[j].input;
    jb.u_begin = (uint32_t)u;
    u += (long)((jobs[j].N + 127) / 128) * jb.n_kb;
  }
  for (int j = n_jobs; j < MAX_JOBS; ++j) p.jobs[j] = p.jobs[0];
  if (u > (long)(0xFFFFFFFFu / (MAX_GRID + 1))) return HBL_ERR_TOO_LARGE;   // the kernel indexes units in 32 bits
  p.U = (uint32_t)u;
  p.part = part; p.flags = flags;
  p.status = device_status_word();
  if (p.status == nullptr) return HBL_ERR_CUDA;
  p.T = T;
  p.release_early = early_release_reserve >= 0 ? 1 : 0;
  p.ready = ready ? ready->ready : nullptr;
  for (int m = 0; m < MAX_MAPS; ++m) p.ready_target[m] = ready ? ready->target[m] : 0u;
  p.done = (ready && last_pass) ? ready->done : nullptr;
  p.done_early = single_pass ? 1 : 0;
  // Every CTA that shares a row block writes (and the owner reads) 128 x t_pad partial sums.  Use
  // all SMs only when each one streams several times that in weights; otherwise fewer, fatter
  // CTAs (never fewer than one per row block, which shares nothing).
  long grid_l = u < n_sm ? u : n_sm;
  {
    long n_rb_all = 0, packed_bytes = 0;
    for (int j = 0; j < n_jobs; ++j) {
      n_rb_all += (jobs[j].N + 127) / 128;
      packed_bytes += (long)((jobs[j].N + 127) / 128) * 128 * inputs[jobs[j].input].K / 4;
    }
    const long part_bytes = 128L * t_pad * 4;
    long want = packed_bytes / (4 * part_bytes);
    if (want < n_rb_all) want = n_rb_all;
    if (want < grid_l) grid_l = want;
    if (grid_l < 1) grid_l = 1;
  }
  // A grid that deals every CTA the same whole number of row blocks shares no row block: no partial sums, no
  // owner waiting at the end (measured on 148 SMs: the 7B block at 16 tokens 25.9 -> 24.9 us with 128 CTAs, at 256
  // tokens 135 -> 120 us; 4096 -> 12288 at 16 tokens 10.2 -> 9.0 us with 96).  It is taken when it keeps at
  // least 5/8 of the SMs busy; otherwise the ranges stay ragged and every SM gets one.
  {
    long per_rb = 1;                                         // least common multiple of the jobs' units per row block
    for (int j = 0; j < n_jobs && per_rb <= u; ++j) {
      long a = per_rb, b = p.jobs[j].n_kb;
      while (b != 0) { const long t = a % b; a = b; b = t; }
      per_rb = per_rb / a * p.jobs[j].n_kb;
    }
    if (per_rb <= u && u % per_rb == 0) {
      const long groups = u / per_rb;                        // a CTA takes groups / g of them, g a divisor of groups
      for (long m = (groups + grid_l - 1) / grid_l; m <= groups && (groups / m) * 8 >= 5L * n_sm_all; ++m) {
        if (groups % m != 0) continue;
        grid_l = groups / m;
        break;
      }
    }
  }
  const int grid = (int)grid_l;
  if (t_pad == 16) return launch_kbp<16>(kbp, maps, p, grid, s);
  if (t_pad == 32) return launch_kbp<32>(kbp, maps, p, grid, s);
  if (t_pad == 64) return launch_kbp<64>(kbp, maps, p, grid, s);
  return kbp == 2 ? launch_variant<128, 2>(maps, p, grid, s) : launch_variant<128, 1>(maps, p, grid, s);
}

// Up to 512 tokens: the weights stream once per 128 tokens (still far cheaper than expanding them to
// int8 in HBM for the large-batch kernel, whose tiles would also be mostly padding at these sizes).
int launch_gemm_stream_multi(const StreamInput* inputs, int n_inputs, const StreamJob* jobs, int n_jobs, int T,
                             int32_t* part, int* flags, cudaStream_t s, int early_release_reserve,
                             const StreamReady* ready) {
  if (T <= 0 || n_jobs <= 0) return HBL_OK;
  if (T > gemm_stream_max_tokens()) return HBL_ERR_TOO_LARGE;
  if (n_jobs > MAX_JOBS || n_inputs > MAX_MAPS || n_inputs <= 0) return HBL_ERR_SHAPE;
  for (int pass = 0; pass * 128 < T; ++pass) {
    const int t0 = pass * 128, tn = T - t0 < 128 ? T - t0 : 128;
    StreamInput in[MAX_MAPS];
    StreamJob jb[MAX_JOBS];
    for (int m = 0; m < n_inputs; ++m)
      in[m] = {inputs[m].codes + (size_t)t0 * inputs[m].K, inputs[m].scale ? inputs[m].scale + t0 : nullptr,
               inputs[m].codesum + t0, inputs[m].K};
    for (int j = 0; j < n_jobs; ++j) {
      jb[j] = jobs[j];
      if (jb[j].y) jb[j].y += (size_t)t0 * jobs[j].N;
      if (jb[j].acc_out) jb[j].acc_out += (size_t)t0 * jobs[j].N;
    }
    const int rc = launch_gemm_stream_pass(in, n_inputs, jb, n_jobs, tn, part, flags + pass * MAX_GRID, s, early_release_reserve,
                                           ready, (pass + 1) * 128 >= T, T <= 128);
    if (rc != HBL_OK) return rc;
  }
  return HBL_OK;
}

int launch_gemm_stream(const int8_t* codes, const float* scale, const int32_t* codesum, int T, int K,
                       const void* W_packed, int N, const float* alpha, __nv_bfloat16* y,
                       int32_t* acc_out, int32_t* acc_ws, int* counters, cudaStream_t s, int early_release_reserve,
                       const StreamReady* ready) {
  StreamInput in = {codes, scale, codesum, K};
  StreamJob job = {W_packed, alpha, y, acc_out, N, 0};
  return launch_gemm_stream_multi(&in, 1, &job, 1, T, acc_ws, counters, s, early_release_reserve, ready);
}

}  // namespace hbl
