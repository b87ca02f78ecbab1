// Persistent, warp-specialised tcgen05 GEMM engine for sm_100a.
//
//   D[M, N] = A[M, K] * B[N, K]^T      bf16 operands, fp32 accumulation in TMEM
//
// One CTA per SM, 64 + 128 * MB * EW threads:
//   warp 0      TMA producer (one lane): global -> 128B-swizzled shared tiles
//   warp 1      MMA issuer (one lane): tcgen05.mma, accumulators in TMEM
//   then 4 * EW epilogue warps per 128-row block: tcgen05.ld the 128 x BN fp32 block and
//   hand it to `Epi` (a warp may read only the TMEM lane quarter given by warp id % 4).
//   EW = 2 puts two warps on every lane quarter, each with half of the tile's columns: for
//   epilogues whose per-chunk work is a long dependent chain (a single warp per scheduler
//   cannot hide its own latencies) and that keep no state across chunks.
// MB = 1: a 128 x BN tile, accumulator double-buffered in TMEM (2 x BN columns) so the
//   epilogue of tile j overlaps the MMAs of tile j+1; ring slots of (128 x 64) A + (BN x 64) B.
// MB = 2 ("wide"): a 256 x 256 tile as two 128-row blocks that share every B slot (two MMAs
//   per K step), filling all 512 TMEM columns, so the epilogue is not overlapped.  Operand
//   bytes moved from L2 into the SM per flop drop by a third (64 KB per 256x256x64 instead
//   of 48 KB per 128x256x64); measured on B200 that traffic, not the tensor pipe, bounds the
//   sustained rate (under the power cap as well as at full clocks), so the trade pays.
//
// Either operand may be "K-major" (contraction index contiguous in global
// memory: the tensor map's inner dimension is K) or "MN-major" (the M or N index
// contiguous: the tensor map's inner dimension is M/N and its outer one is K).
//
// Work is cut into units: a unit is one 128-row tile and a contiguous range of
// BN-wide column tiles.  The epilogue keeps per-thread state across the tiles of
// a unit (e.g. a running max / sum-exp), which is how the vocabulary reduction
// is fused without ever storing the logits.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

#include "ptx.cuh"

namespace cpmtp {

constexpr int kBM = 128;          // rows per tile = TMEM lanes
constexpr int kBK = 64;           // bf16 elements per 128-byte swizzle row
constexpr int kEpiThreads = 128;   // epilogue threads per 128-row block

// Values raised in the device status word.
constexpr int kDevOk = 0;
constexpr int kDevTargetOutOfRange = 1;
constexpr int kDevWaitTimeout = 2;
constexpr int kDevIndexOutOfRange = 3;   // checked build only, see CPMTP_INDEX_OK

// Checked build (-DCPMTP_DEBUG, libcpmtp_debug.so): every store and every gather of an epilogue first
// compares the element range it is about to touch with the extent of the buffer it addresses.  A range
// that does not fit raises status 3 (in a per-device word that cpmtp_debug_status() reads, and from there
// in the caller's dev_status at the end of the kernel) and the access is skipped; nothing traps.  In the
// release build the macro is the constant `true` and its arguments are not evaluated.
#ifdef CPMTP_DEBUG
__device__ int g_debug_status = 0;
__device__ __forceinline__ bool index_ok(unsigned long long first, unsigned long long count,
                                         unsigned long long extent) {
  if (first + count <= extent && first + count >= first) return true;
  atomicMax(&g_debug_status, kDevIndexOutOfRange);
  return false;
}
#define CPMTP_INDEX_OK(first, count, extent)                                            \
  ::cpmtp::index_ok(static_cast<unsigned long long>(first), static_cast<unsigned long long>(count), \
                    static_cast<unsigned long long>(extent))
#else
#define CPMTP_INDEX_OK(first, count, extent) true
#endif

struct Sched {
  int m_tiles;    // number of (128 * MB)-row tiles
  int n_tiles;    // number of BN-column tiles
  int n_splits;   // column tiles are cut into this many contiguous ranges
  int m_group;    // row tiles that are swept together (L2 locality)
  int k_blocks;   // contraction length / 64, rounded up
  int units;      // ceil(m_tiles / m_group) * m_group * n_splits
  // Segmented columns (0 = off): the B rows form segments of seg_stride rows, each covered by
  // seg_tiles column tiles that start at the segment's first row (the last tile of a segment
  // may run into the next one; the epilogue masks it).  Column tile nt then starts at B row
  // (nt / seg_tiles) * seg_stride + (nt % seg_tiles) * BN instead of nt * BN.
  int seg_tiles;
  int seg_stride;
  // Grouped rows of A (0 = off; K-major A, MB = 1 only): the A tensor map is 3-D [groups][r][K] and a
  // row tile holds a_groups whole groups, each padded to 128 / a_groups rows (see make_grouped_tmap_bf16).
  int a_groups;
  // Longest time (microseconds) any single wait inside the kernel may take before the CTA gives up,
  // raises device status 2 and unwinds.  Set by the launcher.
  unsigned wait_limit_us;
  // Test hook for that give-up path (0 = off): the producer of every CTA leaves out the load (and the
  // barrier arrival) of its test_skip_load-th pipeline slot fill, so the consumer's wait for it runs out.
  int test_skip_load;
};

inline Sched make_sched(int m_tiles, int n_tiles, int n_splits, int m_group, int k_blocks) {
  Sched s;
  if (n_splits > n_tiles) n_splits = n_tiles;
  if (n_splits < 1) n_splits = 1;
  if (m_group > m_tiles) m_group = m_tiles;
  if (m_group < 1) m_group = 1;
  s.m_tiles = m_tiles;
  s.n_tiles = n_tiles;
  s.n_splits = n_splits;
  s.m_group = m_group;
  s.k_blocks = k_blocks;
  s.units = ((m_tiles + m_group - 1) / m_group) * m_group * n_splits;
  s.seg_tiles = 0;
  s.seg_stride = 0;
  s.a_groups = 0;
  s.wait_limit_us = 4000000u;
  s.test_skip_load = 0;
  return s;
}

// Unit u -> (row tile, split, column-tile range).  Consecutive units (which run
// concurrently on neighbouring CTAs) walk the row tiles of one group first.
__device__ __forceinline__ bool decode_unit(const Sched& s, int u, int& m_tile, int& split,
                                            int& n_begin, int& n_end) {
  const int per_group = s.m_group * s.n_splits;
  const int g = u / per_group;
  const int rem = u - g * per_group;
  split = rem / s.m_group;
  m_tile = g * s.m_group + (rem - split * s.m_group);
  if (m_tile >= s.m_tiles) return false;
  n_begin = static_cast<int>((static_cast<long long>(split) * s.n_tiles) / s.n_splits);
  n_end = static_cast<int>((static_cast<long long>(split + 1) * s.n_tiles) / s.n_splits);
  return n_end > n_begin;
}

// A_ROWS < 128 ("skinny A", K-major A only): the problem has at most A_ROWS rows, so only
// that many rows of the A tile are fetched and given shared memory; the MMA still spans 128
// rows and the accumulator rows beyond A_ROWS hold garbage that no epilogue may use.  The
// space saved buys deeper pipelining of the B stream (bandwidth-bound draft scoring).
template <int BN_, int STAGES_, bool A_MN_, bool B_MN_, int A_ROWS_ = kBM, int MB_ = 1, int EW_ = 1>
struct TileCfg {
  static constexpr int BN = BN_;
  static constexpr int STAGES = STAGES_;
  static constexpr bool A_MN = A_MN_;
  static constexpr bool B_MN = B_MN_;
  static constexpr int MB = MB_;                       // 128-row blocks per tile
  static constexpr int EW = EW_;                       // epilogue warps per TMEM lane quarter of a row block
  static constexpr int A_ROWS = A_ROWS_;               // rows of A fetched per 128-row block
  static constexpr int TILE_M = kBM * MB;
  static constexpr int A_BLOCK_BYTES = A_ROWS * kBK * 2;
  static constexpr int A_BYTES = A_BLOCK_BYTES * MB;
  static constexpr int ACC_STAGES = MB == 1 ? 2 : 1;
  static constexpr int THREADS = 64 + kEpiThreads * MB * EW;
  static_assert(EW == 1 || (EW == 2 && BN_ % 128 == 0), "column halves are whole 64-column blocks");
  static_assert(MB == 1 || MB == 2, "one or two 128-row blocks");
  static_assert(MB == 1 || (A_ROWS == kBM && BN == 256), "wide tiles are 256 x 256");
  static_assert(A_ROWS == kBM || (!A_MN_ && A_ROWS % 8 == 0 && A_ROWS >= 8), "skinny A needs a K-major A");
  static constexpr int B_BYTES = BN * kBK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int ACC_COLS = BN * MB * ACC_STAGES;
  static constexpr int TMEM_COLS = (ACC_COLS <= 32) ? 32 : (ACC_COLS <= 64) ? 64 : (ACC_COLS <= 128) ? 128
                                   : (ACC_COLS <= 256) ? 256 : 512;
  static_assert(ACC_COLS <= 512, "TMEM has 512 columns");
  static_assert(BN % 16 == 0 && BN >= 16 && BN <= 256, "MMA N must be a multiple of 16 in [16, 256]");
  static_assert(!B_MN || BN % 64 == 0, "an MN-major B tile is loaded in 64-wide boxes");
  static_assert(STAGE_BYTES % 1024 == 0, "stages must keep 1024-byte alignment for the swizzle");
};

constexpr int kBarrierBytes = 256;

template <class Cfg, class Epi>
constexpr int gemm_smem_bytes() {
  return 1024 + Cfg::STAGES * Cfg::STAGE_BYTES + kBarrierBytes + Epi::SMEM_PER_WARP * 4 * Cfg::MB * Cfg::EW;
}

// Shared memory: [<= 1023 B alignment pad][STAGES operand slots][epilogue staging: Epi::SMEM_PER_WARP bytes for each
// of the 4 * MB * EW epilogue warps][barriers].
template <class Cfg, class Epi>
__global__ void __launch_bounds__(Cfg::THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const Sched sched, const __grid_constant__ typename Epi::Params ep, int* __restrict__ dev_status) {
  constexpr int kEpiSmem = Epi::SMEM_PER_WARP * 4 * Cfg::MB * Cfg::EW;
  static_assert(kEpiSmem % 1024 == 0, "epilogue staging keeps the 1024-byte alignment of the slots");
  static_assert(1024 + Cfg::STAGES * Cfg::STAGE_BYTES + kBarrierBytes + kEpiSmem <= 232448,
                "more shared memory than a CTA can have");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = ptx::smem_u32(smem_raw);
  const uint32_t pad = (1024u - (raw_addr & 1023u)) & 1023u;
  uint8_t* smem = smem_raw + pad;
  const uint32_t tiles_addr = raw_addr + pad;
  uint8_t* epi_smem = smem + Cfg::STAGES * Cfg::STAGE_BYTES;
  uint8_t* bar_mem = epi_smem + kEpiSmem;
  const uint32_t bar_addr = tiles_addr + Cfg::STAGES * Cfg::STAGE_BYTES + kEpiSmem;
  // barrier layout (8 bytes each): full[STAGES], empty[STAGES], tfull[2], tempty[2], drain
  auto full_bar = [&](int s) { return bar_addr + 8u * s; };
  auto empty_bar = [&](int s) { return bar_addr + 8u * (Cfg::STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_addr + 8u * (2 * Cfg::STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_addr + 8u * (2 * Cfg::STAGES + 2 + a); };
  const uint32_t drain_bar = bar_addr + 8u * (2 * Cfg::STAGES + 4);
  static_assert(8 * (2 * Cfg::STAGES + 5) + 16 <= kBarrierBytes, "barrier area too small");
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_mem + kBarrierBytes - 16);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_mem + kBarrierBytes - 8);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint64_t wait_ns = static_cast<uint64_t>(sched.wait_limit_us) * 1000ull;

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::STAGES; ++s) {
      ptx::mbar_init(full_bar(s), 1);
      ptx::mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      ptx::mbar_init(tempty_bar(a), kEpiThreads * Cfg::MB * Cfg::EW);
    }
    ptx::mbar_init(drain_bar, 1);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tmap(&tmA);
    ptx::prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_slot)), Cfg::TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // Everything above touched only this CTA's shared memory and TMEM, so it may overlap the tail of the
  // previous kernel in the stream; the operands and outputs may not.
  ptx::grid_dep_wait();

  if (warp == 0) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      int it = 0;
      bool alive = true;
      for (int u = blockIdx.x; u < sched.units && alive; u += gridDim.x) {
        int m_tile, split, n_begin, n_end;
        if (!decode_unit(sched, u, m_tile, split, n_begin, n_end)) continue;
        for (int nt = n_begin; nt < n_end && alive; ++nt) {
          const int b_row0 = sched.seg_tiles > 0
                                 ? (nt / sched.seg_tiles) * sched.seg_stride + (nt % sched.seg_tiles) * Cfg::BN
                                 : nt * Cfg::BN;
          for (int kb = 0; kb < sched.k_blocks; ++kb, ++it) {
            const int s = it % Cfg::STAGES;
            const uint32_t ph = (it / Cfg::STAGES) & 1;
            if (!ptx::mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, wait_ns)) { alive = false; break; }
            if (sched.test_skip_load != 0 && it + 1 == sched.test_skip_load) continue;   // test hook, see Sched
            ptx::mbar_arrive_expect_tx(full_bar(s), Cfg::STAGE_BYTES);
            const uint32_t a_dst = tiles_addr + s * Cfg::STAGE_BYTES;
            const uint32_t b_dst = a_dst + Cfg::A_BYTES;
            if constexpr (!Cfg::A_MN) {
              // one box of A_ROWS * MB rows: block b lands at a_dst + b * A_BLOCK_BYTES
              if (sched.a_groups > 0) {
                ptx::tma_load_3d(a_dst, &tmA, full_bar(s), kb * kBK, 0, m_tile * sched.a_groups);
              } else {
                ptx::tma_load_2d(a_dst, &tmA, full_bar(s), kb * kBK, m_tile * Cfg::TILE_M);
              }
            } else {
#pragma unroll
              for (int j = 0; j < Cfg::TILE_M / 64; ++j)
                ptx::tma_load_2d(a_dst + j * 8192, &tmA, full_bar(s), m_tile * Cfg::TILE_M + j * 64, kb * kBK);
            }
            if constexpr (!Cfg::B_MN) {
              ptx::tma_load_2d(b_dst, &tmB, full_bar(s), kb * kBK, b_row0);
            } else {
#pragma unroll
              for (int j = 0; j < Cfg::BN / 64; ++j)
                ptx::tma_load_2d(b_dst + j * 8192, &tmB, full_bar(s), b_row0 + j * 64, kb * kBK);
            }
          }
        }
      }
      // All of this CTA's operand loads are issued: the next kernel in the stream may be scheduled
      // (its blocks start as SMs free up and do their own set-up before they wait for this grid).
      ptx::grid_dep_launch();
      // Drain: every load issued must have landed before this CTA's shared memory is released.
      const int issued = it;
      for (int back = 1; back <= Cfg::STAGES && back <= issued; ++back) {
        const int j = issued - back;
        ptx::mbar_wait(full_bar(j % Cfg::STAGES), (j / Cfg::STAGES) & 1, abort_flag, wait_ns, false);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(kBM, Cfg::BN, Cfg::A_MN ? 1 : 0, Cfg::B_MN ? 1 : 0);
      constexpr uint32_t a_kstep = Cfg::A_MN ? 2048u : 32u;   // bytes per 16-element K step
      constexpr uint32_t b_kstep = Cfg::B_MN ? 2048u : 32u;
      // K-major: 8-row groups are 1024 B apart (stride offset); the leading offset is unused.
      // MN-major: 64-element blocks along M/N are 8192 B apart (leading offset), 8-row K groups 1024 B.
      constexpr uint32_t a_lbo = Cfg::A_MN ? 8192u : 16u;
      constexpr uint32_t b_lbo = Cfg::B_MN ? 8192u : 16u;
      int it = 0, acc_it = 0;
      bool alive = true;
      for (int u = blockIdx.x; u < sched.units && alive; u += gridDim.x) {
        int m_tile, split, n_begin, n_end;
        if (!decode_unit(sched, u, m_tile, split, n_begin, n_end)) continue;
        for (int nt = n_begin; nt < n_end && alive; ++nt, ++acc_it) {
          const int acc = acc_it % Cfg::ACC_STAGES;
          const uint32_t acc_ph = (acc_it / Cfg::ACC_STAGES) & 1;
          if (!ptx::mbar_wait(tempty_bar(acc), acc_ph ^ 1u, abort_flag, wait_ns)) { alive = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t d_tmem = tmem_base + acc * Cfg::BN * Cfg::MB;
          for (int kb = 0; kb < sched.k_blocks; ++kb, ++it) {
            const int s = it % Cfg::STAGES;
            const uint32_t ph = (it / Cfg::STAGES) & 1;
            if (!ptx::mbar_wait(full_bar(s), ph, abort_flag, wait_ns)) { alive = false; break; }
            ptx::tc_fence_after_sync();
            const uint32_t a_src = tiles_addr + s * Cfg::STAGE_BYTES;
            const uint32_t b_src = a_src + Cfg::A_BYTES;
#pragma unroll
            for (int kk = 0; kk < kBK / 16; ++kk) {
              const uint64_t bdesc = ptx::make_smem_desc_sw128(b_src + kk * b_kstep, b_lbo, 1024);
#pragma unroll
              for (int mb = 0; mb < Cfg::MB; ++mb) {
                const uint64_t adesc =
                    ptx::make_smem_desc_sw128(a_src + mb * Cfg::A_BLOCK_BYTES + kk * a_kstep, a_lbo, 1024);
                ptx::umma_bf16(d_tmem + mb * Cfg::BN, adesc, bdesc, idesc, (kb | kk) != 0 ? 1u : 0u);
              }
            }
            ptx::umma_commit(empty_bar(s));   // frees the slot once these MMAs have read it
          }
          if (alive) ptx::umma_commit(tfull_bar(acc));
        }
      }
      // Drain: all issued MMAs must retire before TMEM is freed.
      ptx::umma_commit(drain_bar);
      ptx::mbar_wait(drain_bar, 0, abort_flag, wait_ns, false);
    }
  } else {
    // ------------------------------------------------------------ epilogue
    // These waits ignore the other roles' abort flag: all four warps wait on the
    // same barrier, so they either all pass or all time out, and no warp is left
    // alone at a barrier an epilogue might use internally.
    const int quarter = warp & 3;                 // TMEM lane quarter this warp may read
    const int wgroup = (warp - 2) >> 2;           // group of four warps: one row block, one column part
    const int mblock = wgroup % Cfg::MB;          // which 128-row block of the tile
    const int cpart = wgroup / Cfg::MB;           // which part of the tile's columns (EW > 1)
    const int row_in_tile = quarter * 32 + lane;  // row within that block
    const int epi_tid = (threadIdx.x - 64) & (kEpiThreads - 1);
    uint8_t* my_smem = epi_smem + wgroup * (Epi::SMEM_PER_WARP * 4);   // this warp group's staging
    typename Epi::State st;
    int acc_it = 0;
    bool alive = true;
    for (int u = blockIdx.x; u < sched.units && alive; u += gridDim.x) {
      int m_tile, split, n_begin, n_end;
      if (!decode_unit(sched, u, m_tile, split, n_begin, n_end)) continue;
      const int m_block_tile = m_tile * Cfg::MB + mblock;   // index of this warp's 128-row block
      Epi::unit_begin(ep, st, m_block_tile, split, row_in_tile);
      for (int nt = n_begin; nt < n_end; ++nt, ++acc_it) {
        const int acc = acc_it % Cfg::ACC_STAGES;
        const uint32_t acc_ph = (acc_it / Cfg::ACC_STAGES) & 1;
        Epi::pre_tile(ep, st, m_block_tile, nt, row_in_tile);
        if (!ptx::mbar_wait(tfull_bar(acc), acc_ph, abort_flag, wait_ns, false)) { alive = false; break; }
        ptx::tc_fence_after_sync();
        const uint32_t tacc = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                              (acc * Cfg::MB + mblock) * Cfg::BN;
        if constexpr (Cfg::EW == 1) {
          Epi::tile(ep, st, tacc, m_block_tile, nt, row_in_tile, my_smem, epi_tid);
        } else {
          constexpr int kPart = Cfg::BN / Cfg::EW;
          Epi::tile_part(ep, st, tacc, m_block_tile, nt, row_in_tile, my_smem, epi_tid, cpart * kPart, (cpart + 1) * kPart);
        }
        ptx::tc_fence_before_sync();
        ptx::mbar_arrive(tempty_bar(acc));
      }
      if (alive) Epi::unit_end(ep, st, m_block_tile, split, row_in_tile, my_smem, epi_tid);
    }
    Epi::role_end(ep, st, my_smem, epi_tid);   // e.g. wait for this thread's asynchronous stores
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  if (warp == 1) ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
  if (threadIdx.x == 0 && *abort_flag != 0 && dev_status != nullptr) atomicMax(dev_status, kDevWaitTimeout);
#ifdef CPMTP_DEBUG
  if (threadIdx.x == 0 && dev_status != nullptr) {
    const int seen = *const_cast<volatile int*>(&g_debug_status);
    if (seen != 0) atomicMax(dev_status, seen);
  }
#endif
}

}  // namespace cpmtp
