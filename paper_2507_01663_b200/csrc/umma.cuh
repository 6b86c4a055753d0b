// Blackwell (sm_100a) building blocks: mbarrier, TMA tile loads, tcgen05 MMA with TMEM
// accumulators -- inline PTX only -- and the warp-specialised persistent GEMM main loop every
// tensor-core kernel of the library is built on.
//
//   C[M,N] = sum_k A(m,k) * B(n,k)    A, B bf16; fp32 accumulation in tensor memory; the epilogue
//   functor consumes the accumulator tile.  Each operand is either K-major (stored [rows, K], K
//   contiguous) or MN-major (stored [K, rows], the M or N index contiguous), chosen at compile
//   time, so products with a transposed operand need no transposed copy.
//
// CTA = 6 warps.  warp 0: TMA producer (one elected lane).  warp 1: allocates TMEM and issues
// tcgen05.mma (one elected lane).  warps 2-5: epilogue, one TMEM lane (= output row) per thread.
// Shared memory holds a ring of kStages {A 128x64, B 256x64} bf16 tiles in the 128-byte swizzle
// TMA writes and the MMA descriptors expect; TMEM holds two 128x256 fp32 accumulators so the
// epilogue of tile i overlaps the MMAs of tile i+1.
//
// Every wait is bounded: a wait that exceeds kWaitLimitNs raises AF_DEVERR_WATCHDOG, makes all
// roles leave their loops, frees TMEM and returns.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace af {
namespace umma {

constexpr int kBM = 128;          // rows of A per tile  (UMMA M)
constexpr int kBN = 256;          // rows of B per tile  (UMMA N)
constexpr int kBK = 64;           // K elements per stage = one 128-byte swizzle row
constexpr int kUmmaK = 16;        // K per tcgen05.mma for 16-bit inputs
constexpr int kStages = 4;
constexpr int kABytes = kBM * kBK * 2;
constexpr int kBBytes = kBN * kBK * 2;
constexpr int kStageBytes = kABytes + kBBytes;            // 48 KB
constexpr int kTmemCols = 512;                            // 2 accumulators x 256 fp32 columns
constexpr int kThreads = 192;
constexpr int kEpiThreads = 128;
constexpr int kMnBoxBytes = 64 * kBK * 2;                 // one 64 (MN) x 64 (K) box of an MN-major tile
constexpr int kEpiStageBytes = 4096;                      // per epilogue warp: a 32 x 32 fp32 chunk
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int kSmemBytesStaged = kSmemBytes + 4 * kEpiStageBytes;
constexpr unsigned long long kWaitLimitNs = 4000000000ull;
constexpr unsigned int kWatchdogBit = 2u;                 // AF_DEVERR_WATCHDOG

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the CTA is aborting (some wait ran out of time).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned long long limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 63u) == 0u) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > limit_ns) { *abort_flag = 1; return false; }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst_smem, const CUtensorMap* map, uint32_t bar,
                                            int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst_smem), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, 128 x 256 x 16, bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void mma_bf16_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                            uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrive on `bar` once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor for a K-major bf16 tile stored as rows of 128 bytes with the
// 128-byte swizzle (what TMA writes for a 64-element-wide box): 8-row groups are 1024 bytes
// apart (stride byte offset), the leading byte offset is unused for this layout.
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);  // start address, 16-byte units
  d |= (uint64_t)1 << 16;                        // leading byte offset (ignored when swizzled)
  d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset
  d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                        // layout: 128-byte swizzle
  return d;
}
// Descriptor for an MN-major bf16 tile: TMA writes it as boxes of 64 K-rows x 128 bytes (64
// consecutive M or N indices), 128-byte swizzle, one box per 64 indices.  Inside a box, groups of
// 8 K-rows are 1024 bytes apart (stride byte offset); boxes are kMnBoxBytes apart (leading byte
// offset).  One MMA (K = 16) spans two 8-row groups, so the K step is 2048 bytes.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(kMnBoxBytes >> 4) << 16;       // leading byte offset: next 64 M/N indices
  d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset: next 8 K-rows
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor: D fp32, A and B bf16, M x N tile, each operand K-major or MN-major.
__host__ __device__ constexpr uint32_t instr_desc_bf16_f32(int m, int n, bool a_mn = false, bool b_mn = false) {
  return (1u << 4)                         // D format: fp32
         | (1u << 7) | (1u << 10)          // A, B format: bf16
         | ((a_mn ? 1u : 0u) << 15)        // A major: 0 = K, 1 = MN
         | ((b_mn ? 1u : 0u) << 16)        // B major
         | ((uint32_t)(n >> 3) << 17)      // N / 8
         | ((uint32_t)(m >> 4) << 24);     // M / 16
}

// ------------------------------------------------------------------------------------------
// Work decomposition shared by all three roles.
// A unit is one token/row tile (m_tile) times a contiguous range of B tiles (split s of S);
// CTA b processes units b, b + grid, b + 2 grid, ...  Consecutive units share the m_tile, so
// the CTAs running at one time work on grid/S row tiles and sweep the B tiles together: the
// A panels stay L2-resident and every B tile is fetched from HBM once per wave.
// ------------------------------------------------------------------------------------------
struct GemmShape {
  int M, N, K;          // logical extents (rows of A, rows of B, reduction length)
  int m_tiles, n_tiles; // ceil(M/128), ceil(N/256)
  int splits;           // S: n-tile ranges per m_tile
  int k_blocks;         // ceil(K/64)
  int die0_pairs;       // pair kernel only: > 0 = deal the row tiles by die; the number of CTA pairs the first die hosts
  int die0_rows;        // ... and the number of row tiles (the first ones) those pairs share among themselves
};
__device__ __forceinline__ int split_begin(const GemmShape& g, int s) {
  return (int)(((long long)g.n_tiles * s) / g.splits);
}

// The epilogue functor E provides:
//   struct Params;  struct State;  static constexpr bool kStaged;
//   static __device__ void unit_begin(State&, const Params&, int row, int m_tile, int split);
//   static __device__ void chunk(State&, const Params&, int row, int col0, const uint32_t (&v)[32],
//                                uint8_t* stage);
//        -- 32 fp32 accumulator columns col0 .. col0+31 of output row `row` (bit patterns); called
//           by all 32 lanes of an epilogue warp together (lane L holds row row0 + L).  `stage` is
//           the warp's private kEpiStageBytes of shared memory (kStaged only, else null), used to
//           turn row-per-lane data into coalesced global stores.
//   static __device__ void unit_end(State&, const Params&, int row, int split);
template <class E, bool kAMN = false, bool kBMN = false>
__global__ void __launch_bounds__(kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
            const GemmShape g, const typename E::Params ep, unsigned int* d_err) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;                 // 1024-byte aligned tile ring
  const uint32_t bars = tiles + kStages * kStageBytes;           // barriers behind the ring
  // barrier addresses
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (kStages + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * kStages + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * kStages + 2 + a); };
  const uint32_t tmem_slot = bars + 8u * (2 * kStages + 4);
  uint8_t* const epi_stage_base = smem_raw + (bars + 256u - raw);   // behind the barrier block
  volatile uint32_t* tmem_slot_ptr =
      reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - raw));
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), kEpiThreads); }
    fence_mbar_init();
    tma_prefetch_desc(&tmap_a);
    tma_prefetch_desc(&tmap_b);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;

  const int total_units = g.m_tiles * g.splits;

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0; bool ok = true;
      for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
        const int m_tile = u / g.splits, s = u % g.splits;
        const int nb = split_begin(g, s), ne = split_begin(g, s + 1);
        for (int nt = nb; nt < ne && ok; ++nt) {
          for (int kb = 0; kb < g.k_blocks; ++kb) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, &abort_flag)) { ok = false; break; }
            const uint32_t a_dst = tiles + stage * kStageBytes;
            mbar_arrive_expect_tx(full_bar(stage), kStageBytes);
            if constexpr (kAMN) {
#pragma unroll
              for (int b = 0; b < kBM / 64; ++b)
                tma_load_2d(a_dst + b * kMnBoxBytes, &tmap_a, full_bar(stage), m_tile * kBM + b * 64, kb * kBK);
            } else {
              tma_load_2d(a_dst, &tmap_a, full_bar(stage), kb * kBK, m_tile * kBM);
            }
            if constexpr (kBMN) {
#pragma unroll
              for (int b = 0; b < kBN / 64; ++b)
                tma_load_2d(a_dst + kABytes + b * kMnBoxBytes, &tmap_b, full_bar(stage), nt * kBN + b * 64, kb * kBK);
            } else {
              tma_load_2d(a_dst + kABytes, &tmap_b, full_bar(stage), kb * kBK, nt * kBN);
            }
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_bf16_f32(kBM, kBN, kAMN, kBMN);
      // descriptor advance per K = 16 step, in 16-byte units: 32 bytes inside a swizzled K-major
      // row, two 8-row groups (2048 bytes) for an MN-major tile
      constexpr uint64_t a_step = kAMN ? (2048 >> 4) : 2, b_step = kBMN ? (2048 >> 4) : 2;
      int stage = 0; uint32_t phase = 0; uint32_t tile_count = 0; bool ok = true;
      for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
        const int s = u % g.splits;
        const int nb = split_begin(g, s), ne = split_begin(g, s + 1);
        for (int nt = nb; nt < ne && ok; ++nt, ++tile_count) {
          const uint32_t acc = tile_count & 1u, acc_phase = (tile_count >> 1) & 1u;
          if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, &abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + acc * kBN;
          for (int kb = 0; kb < g.k_blocks; ++kb) {
            if (!mbar_wait(full_bar(stage), phase, &abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = tiles + stage * kStageBytes;
            const uint64_t a_desc = kAMN ? smem_desc_mn_sw128(a_addr) : smem_desc_k_sw128(a_addr);
            const uint64_t b_desc = kBMN ? smem_desc_mn_sw128(a_addr + kABytes) : smem_desc_k_sw128(a_addr + kABytes);
#pragma unroll
            for (int k = 0; k < kBK / kUmmaK; ++k) {
              mma_bf16_ss(d_tmem, a_desc + (uint64_t)k * a_step, b_desc + (uint64_t)k * b_step, idesc,
                          (kb | k) != 0 ? 1u : 0u);
            }
            mma_commit(empty_bar(stage));  // smem slot reusable once these MMAs have read it
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (ok) mma_commit(tfull_bar(acc));  // accumulator complete
        }
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue (warps 2..5)
    const int quarter = warp & 3;                       // TMEM lanes this warp may touch
    const int row_in_tile = quarter * 32 + lane;
    uint32_t tile_count = 0; bool ok = true;
    typename E::State st;
    uint8_t* const stage = E::kStaged ? epi_stage_base + (warp - 2) * kEpiStageBytes : nullptr;
    for (int u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
      const int m_tile = u / g.splits, s = u % g.splits;
      const int nb = split_begin(g, s), ne = split_begin(g, s + 1);
      const int row = m_tile * kBM + row_in_tile;
      E::unit_begin(st, ep, row, m_tile, s);
      for (int nt = nb; nt < ne && ok; ++nt, ++tile_count) {
        const uint32_t acc = tile_count & 1u, acc_phase = (tile_count >> 1) & 1u;
        // the lanes of a warp must leave together: chunk() may synchronise the warp
        if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), acc_phase, &abort_flag))) { ok = false; break; }
        tc_fence_after();
        const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * kBN;
#pragma unroll 1
        for (int c = 0; c < kBN / 32; ++c) {
          uint32_t v[32];
          tmem_ld32(t_row + c * 32, v);
          tmem_ld_wait();
          E::chunk(st, ep, row, nt * kBN + c * 32, v, stage);
        }
        tc_fence_before();
        mbar_arrive(tempty_bar(acc));
      }
      if (ok) E::unit_end(st, ep, row, s);
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && abort_flag) atomicOr(d_err, kWatchdogBit);
  if (warp == 1) {
    if (abort_flag) __nanosleep(1000000);  // let copies in flight land before the CTA retires
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}


// ==========================================================================================
// CTA-pair variant (cta_group::2).  Two CTAs of a cluster, on the two SMs of one pair, compute a
// 256 x 256 tile together: each holds 128 rows of A and 128 of the 256 rows of B in its own
// shared memory and 128 rows of the fp32 accumulator in its own tensor memory; one thread of the
// pair's first CTA (the leader) issues every MMA for both.  Per 128 x 256 x 64 block of work a SM
// now stages 32 KB instead of 48 KB, which deepens the ring to 6 stages and takes a third off the
// L2 -> shared-memory traffic.
//
// Barriers (same shared-memory offsets in both CTAs):
//   full[s]   leader's copy only: one arrival (the leader's producer, with the byte count of both
//             CTAs' copies); each CTA's TMA loads complete on it.
//   empty[s]  per CTA: the leader's MMA thread commits to both copies at once.
//   tfull[a]  per CTA: accumulator a complete (committed to both copies at once).
//   tempty[a] leader's copy only: one arrival per epilogue warp of either CTA (8 in all).
// No load is multicast; every CTA fetches its own operand halves.  The leaders' producers pace
// one another with a tile clock in global memory (a counter the host zeroes before the launch).
// ==========================================================================================
constexpr int kPairBM = 256;                                  // rows of A per pair tile
constexpr int kPairStages = 6;
constexpr unsigned int kClockWindow = 1;                      // ticks a pair may start ahead of the slowest pair
constexpr int kClockTickKBlocks = 64;                         // K blocks per tick when a tile has more than 96
constexpr unsigned long long kClockPatienceNs = 200000ull;    // longest single wait on the tile clock,
constexpr unsigned long long kClockPatiencePerKBlockNs = 2000ull;  // plus this per K block of a tick (~5 tick times)
constexpr unsigned int kClockRestTicks = 16;                  // ticks a pair goes unpaced after a wait that ran out
constexpr int kClockQuickRetries = 8;                         // waits in a row that may run out before the rests double
constexpr int kPairBBytes = (kBN / 2) * kBK * 2;              // this CTA's half of the B tile
constexpr int kPairStageBytes = kABytes + kPairBBytes;        // 32 KB
constexpr int kPairSmemBytes = kPairStages * kPairStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int kPairSmemBytesStaged = kPairSmemBytes + 4 * kEpiStageBytes;

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on the barrier at the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar, uint32_t rank) {
  asm volatile(
      "{\n\t.reg .b32 ra;\n\t"
      "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
      "mbarrier.arrive.release.cluster.shared::cluster.b64 _, [ra];\n\t}"
      ::"r"(bar), "r"(rank) : "memory");
}
// Cluster-wide address of the shared-memory location `addr` of CTA `rank`.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
// TMA tile load of a CTA pair: data lands in this CTA's shared memory, the bytes are counted on
// `leader_bar`, a barrier of the pair's leader given by its cluster-wide address.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst_smem, const CUtensorMap* map,
                                                 uint32_t leader_bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst_smem), "l"(map), "r"(leader_bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem of both CTAs] (+)= A * B^T, 256 x 256 x 16 over the pair.
__device__ __forceinline__ void mma_bf16_ss_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                                 uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrive on `bar` in both CTAs of the pair once every MMA issued so far has completed.
__device__ __forceinline__ void mma_commit_pair(uint32_t bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((unsigned short)3) : "memory");
}

__device__ __forceinline__ uint32_t ld_shared_cluster_u32(uint32_t cluster_addr) {
  uint32_t v;
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(cluster_addr) : "memory");
  return v;
}

// Which units a pair processes.  Plain dealing: the pair of rank r takes units r, r + n_pairs, ...
// (unit u = row tile u / S, vocabulary range u % S).  Die-aware dealing: the B200 is two dies, each
// with its own half of L2, and a line that SMs of both dies read is kept in both halves; the A panel
// of a row tile therefore costs L2 space twice when the pairs working on its S ranges sit on
// different dies.  Here ranks [0, n0) -- the pairs that run on the first die, which they learn from a
// measured table of SM ids -- share the first rows0 row tiles among themselves and the other ranks
// the rest, so a panel lives in one half of L2 only.  Ranks are handed out by atomic counters and are
// a permutation of 0 .. n_pairs - 1 whatever the table says, so every unit is processed exactly once in
// either mode; only the cache behaviour depends on the table being right.
struct PairWork {
  int first, step, end, base_unit;     // units base_unit + first, base_unit + first + step, ... below base_unit + end
};
__host__ __device__ __forceinline__ PairWork pair_work(const GemmShape& g, int rank, int n_pairs) {
  const int total = g.m_tiles * g.splits;
  const int n0 = g.die0_pairs, n1 = n_pairs - n0;
  if (n0 <= 0 || n1 <= 0) return PairWork{rank, n_pairs, total, 0};
  const int rows0 = g.die0_rows;                 // chosen by the host: in proportion to the pairs, rounds balanced
  if (rank < n0) return PairWork{rank, n0, rows0 * g.splits, 0};
  return PairWork{rank - n0, n1, (g.m_tiles - rows0) * g.splits, rows0 * g.splits};
}
// most units any pair processes in this launch
__device__ __forceinline__ int pair_work_most(const GemmShape& g, int n_pairs) {
  const PairWork a = pair_work(g, 0, n_pairs), b = pair_work(g, n_pairs - 1, n_pairs);
  const int ua = (a.end + a.step - 1) / a.step, ub = (b.end + b.step - 1) / b.step;
  return ua > ub ? ua : ub;
}

// Work decomposition of the pair kernel: a unit is one 256-row tile times a range of B tiles;
// see PairWork for which units a pair processes.
template <class E, bool kAMN = false, bool kBMN = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                 const GemmShape g, const typename E::Params ep, unsigned int* d_err, unsigned int* tile_clock,
                 unsigned int* die_counters, const unsigned char* die_of_sm) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;
  const uint32_t bars = tiles + kPairStages * kPairStageBytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (kPairStages + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * kPairStages + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * kPairStages + 2 + a); };
  const uint32_t tmem_slot = bars + 8u * (2 * kPairStages + 4);
  uint8_t* const epi_stage_base = smem_raw + (bars + 256u - raw);
  volatile uint32_t* tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - raw));
  __shared__ int abort_flag;
  __shared__ uint32_t s_pair_rank;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader
  const int n_pairs = gridDim.x >> 1;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < kPairStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8); }
    fence_mbar_init();
    tma_prefetch_desc(&tmap_a);
    tma_prefetch_desc(&tmap_b);
    // The pair's rank in the work assignment.  With die-aware dealing the leader looks its SM up in
    // the table and takes the next rank of that die from the die's counter (the host zeroed both);
    // should the die already be full -- a table that does not match where the pairs really run -- it
    // takes one of the other die's: n_pairs claimants for n0 + n1 = n_pairs ranks, so that always works.
    uint32_t r = (uint32_t)(blockIdx.x >> 1);
    if (rank == 0 && g.die0_pairs > 0 && g.die0_pairs < n_pairs && die_counters != nullptr && die_of_sm != nullptr) {
      uint32_t smid;
      asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
      const uint32_t n0 = (uint32_t)g.die0_pairs, n1 = (uint32_t)n_pairs - n0;
      uint32_t die = smid < 256u ? (uint32_t)die_of_sm[smid] & 1u : 0u;
      uint32_t idx = atomicAdd(die_counters + die, 1u);
      if (idx >= (die ? n1 : n0)) {
        die ^= 1u;
        idx = atomicAdd(die_counters + die, 1u);
        if (idx >= (die ? n1 : n0)) { abort_flag = 1; idx = 0; }     // cannot happen; never run with a duplicate rank
      }
      r = die ? n0 + idx : idx;
    }
    s_pair_rank = r;
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();       // the peer's barriers exist before anything is signalled across CTAs
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;
  // both CTAs work from the leader's rank
  const int pair = (int)ld_shared_cluster_u32(map_to_cta(smem_u32(&s_pair_rank), 0));
  const PairWork work = pair_work(g, pair, n_pairs);  // m_tiles counts 256-row tiles here

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0; bool ok = true;
      const uint32_t leader_full0 = map_to_cta(full_bar(0), 0);
      // Pacing clock.  Every pair does the same work per K block, so "K blocks issued" measures
      // progress across pairs; a tick is one tile's worth of K blocks, or kClockTickKBlocks of them
      // when tiles are long (the backward's products run thousands of K blocks per tile, and pairs
      // that only met at tile starts drifted far enough apart to lose each other's tiles in L2).
      // The clock counts ticks over all pairs; a pair starts tick j only when all have started tick
      // j - kClockWindow.  It is a hint, not a dependency: a pair that waits longer than its patience
      // goes on without the others for kClockRestTicks ticks (still counting its own), then waits
      // again.  A pair that was held up for a while (one launch in a few hundred sees some SMs
      // stall for a fraction of a millisecond) is caught up with that way, `patience` at a time;
      // before, the pairs left the clock for the rest of the launch and a single stall cost a
      // 200 ms launch 40 ms.  Waits that keep running out (pairs that are not co-resident) are
      // spaced further and further apart.
      unsigned int my_ticks = 0;
      unsigned int skip_until = 0;                                  // no waiting before this tick
      int misses = 0;                                               // waits in a row that ran out
      const bool clock_on = tile_clock != nullptr && rank == 0;
      const int tick_len = g.k_blocks <= 96 ? g.k_blocks : kClockTickKBlocks;
      int to_next_tick = 0;                                         // K blocks until the next tick
      const unsigned long long patience = kClockPatienceNs + kClockPatiencePerKBlockNs * (unsigned long long)tick_len;
      // most ticks any pair starts in this launch
      const unsigned long long most_kb = (unsigned long long)pair_work_most(g, n_pairs) *
                                         (unsigned long long)((g.n_tiles + g.splits - 1) / g.splits) *
                                         (unsigned long long)g.k_blocks;
      const unsigned int clock_most = (unsigned int)((most_kb + tick_len - 1) / tick_len);
      for (int q = work.first; q < work.end && ok; q += work.step) {
        const int u = work.base_unit + q;
        const int m_tile = u / g.splits, s = u % g.splits;
        const int nb = split_begin(g, s), ne = split_begin(g, s + 1);
        const int m0 = m_tile * kPairBM + (int)rank * kBM;          // this CTA's 128 rows of A
        for (int nt = nb; nt < ne && ok; ++nt) {
          const int n0 = nt * kBN + (int)rank * (kBN / 2);          // this CTA's 128 rows of B
          for (int kb = 0; kb < g.k_blocks; ++kb) {
            if (clock_on && to_next_tick-- == 0) {
              to_next_tick = tick_len - 1;
              if (my_ticks >= kClockWindow && my_ticks >= skip_until) {
                const unsigned int need = (unsigned int)n_pairs * (my_ticks - kClockWindow + 1);
                const unsigned long long t0 = globaltimer_ns();
                unsigned int seen;
                bool ran_out = false;
                for (;;) {
                  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(tile_clock) : "memory");
                  if (seen >= need) break;
                  if (globaltimer_ns() - t0 > patience) { ran_out = true; break; }
                  __nanosleep(100);
                }
                if (ran_out) {
                  ++misses;
                  const int doublings = misses <= kClockQuickRetries ? 0 : (misses - kClockQuickRetries < 16 ? misses - kClockQuickRetries : 16);
                  skip_until = my_ticks + (kClockRestTicks << doublings);
                } else {
                  misses = 0;
                }
              }
              atomicAdd(tile_clock, 1u);
              ++my_ticks;
            }
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, &abort_flag)) { ok = false; break; }
            const uint32_t a_dst = tiles + stage * kPairStageBytes;
            const uint32_t lbar = leader_full0 + 8u * stage;
            if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), 2 * kPairStageBytes);
            if constexpr (kAMN) {
#pragma unroll
              for (int b = 0; b < kBM / 64; ++b)
                tma_load_2d_pair(a_dst + b * kMnBoxBytes, &tmap_a, lbar, m0 + b * 64, kb * kBK);
            } else {
              tma_load_2d_pair(a_dst, &tmap_a, lbar, kb * kBK, m0);
            }
            if constexpr (kBMN) {
#pragma unroll
              for (int b = 0; b < kBN / 128; ++b)
                tma_load_2d_pair(a_dst + kABytes + b * kMnBoxBytes, &tmap_b, lbar, n0 + b * 64, kb * kBK);
            } else {
              tma_load_2d_pair(a_dst + kABytes, &tmap_b, lbar, kb * kBK, n0);
            }
            if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
      // a pair that runs out of work counts as having started every remaining tick
      if (clock_on && clock_most > my_ticks) atomicAdd(tile_clock, clock_most - my_ticks);
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (leader only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = instr_desc_bf16_f32(kPairBM, kBN, kAMN, kBMN);
      constexpr uint64_t a_step = kAMN ? (2048 >> 4) : 2, b_step = kBMN ? (2048 >> 4) : 2;
      int stage = 0; uint32_t phase = 0; uint32_t tile_count = 0; bool ok = true;
      for (int q = work.first; q < work.end && ok; q += work.step) {
        const int s = (work.base_unit + q) % g.splits;
        const int nb = split_begin(g, s), ne = split_begin(g, s + 1);
        for (int nt = nb; nt < ne && ok; ++nt, ++tile_count) {
          const uint32_t acc = tile_count & 1u, acc_phase = (tile_count >> 1) & 1u;
          if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, &abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + acc * kBN;
          for (int kb = 0; kb < g.k_blocks; ++kb) {
            if (!mbar_wait(full_bar(stage), phase, &abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = tiles + stage * kPairStageBytes;
            const uint64_t a_desc = kAMN ? smem_desc_mn_sw128(a_addr) : smem_desc_k_sw128(a_addr);
            const uint64_t b_desc = kBMN ? smem_desc_mn_sw128(a_addr + kABytes) : smem_desc_k_sw128(a_addr + kABytes);
#pragma unroll
            for (int k = 0; k < kBK / kUmmaK; ++k) {
              mma_bf16_ss_pair(d_tmem, a_desc + (uint64_t)k * a_step, b_desc + (uint64_t)k * b_step, idesc,
                               (kb | k) != 0 ? 1u : 0u);
            }
            mma_commit_pair(empty_bar(stage));   // both CTAs' slots reusable once these MMAs have read them
            if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
          }
          if (ok) mma_commit_pair(tfull_bar(acc));  // accumulator complete in both CTAs
        }
      }
    }
    __syncwarp();
  } else {
    // ---------------------------------------------------------------- epilogue (warps 2..5, both CTAs)
    const int quarter = warp & 3;
    const int row_in_tile = (int)rank * kBM + quarter * 32 + lane;
    uint32_t tile_count = 0; bool ok = true;
    typename E::State st;
    uint8_t* const stage = E::kStaged ? epi_stage_base + (warp - 2) * kEpiStageBytes : nullptr;
    for (int q = work.first; q < work.end && ok; q += work.step) {
      const int u = work.base_unit + q;
      const int m_tile = u / g.splits, s = u % g.splits;
      const int nb = split_begin(g, s), ne = split_begin(g, s + 1);
      const int row = m_tile * kPairBM + row_in_tile;
      E::unit_begin(st, ep, row, m_tile, s);
      for (int nt = nb; nt < ne && ok; ++nt, ++tile_count) {
        const uint32_t acc = tile_count & 1u, acc_phase = (tile_count >> 1) & 1u;
        if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), acc_phase, &abort_flag))) { ok = false; break; }
        tc_fence_after();
        const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * kBN;
#pragma unroll 1
        for (int c = 0; c < kBN / 32; ++c) {
          uint32_t v[32];
          tmem_ld32(t_row + c * 32, v);
          tmem_ld_wait();
          E::chunk(st, ep, row, nt * kBN + c * 32, v, stage);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(tempty_bar(acc), 0);   // one arrival per warp, on the leader
      }
      if (ok) E::unit_end(st, ep, row, s);
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && abort_flag) atomicOr(d_err, kWatchdogBit);
  if (abort_flag) __nanosleep(1000000);  // let copies in flight land before the CTA retires
  cluster_sync_all();   // neither CTA leaves while the other may still touch its memory or barriers
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

}  // namespace umma
}  // namespace af
