// Epilogues plugged into the tcgen05 GEMM engine.  Each one consumes a
// 128 x BN fp32 accumulator block straight from TMEM; thread `row_in_tile` owns
// one accumulator row and walks it in 32-column chunks.
//
// Interface (static members; smem = the row block's staging area of 4 * SMEM_PER_WARP bytes,
// tid = 0..127 within the row block):
//   unit_begin(params, state, m_tile, split, row)  before the first tile of a work unit
//   pre_tile(params, state, m_tile, n_tile, row)   before the wait for the tile's accumulator:
//                                                  the place for loads that do not depend on it
//   tile(params, state, tacc, m_tile, n_tile, row, smem, tid)
//   unit_end(params, state, m_tile, split, row, smem, tid)
//   role_end(params, state, smem, tid)             once, after the thread's last unit
#pragma once
#include <cstdint>

#include "ptx.cuh"
#include "tc_gemm.cuh"

namespace cpmtp {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct EpiDefaults {
  static constexpr int SMEM_PER_WARP = 0;
  template <class P, class S>
  __device__ static void pre_tile(const P&, S&, int, int, int) {}
  template <class P, class S>
  __device__ static void role_end(const P&, S&, uint8_t*, int) {}
};

// Walk the 32-column chunks at column offsets [c_lo, c_hi) of an accumulator block (multiples of
// 32), calling f(c, v) with the chunk's 32 values of this thread's row.  The TMEM load of the next
// chunk is in flight while f works on the current one (two register arrays in turn), so the load
// latency is paid once per tile instead of once per chunk.
template <class F>
__device__ __forceinline__ void for_each_chunk(uint32_t tacc, int c_lo, int c_hi, F&& f) {
  if (c_lo >= c_hi) return;
  float va[32], vb[32];
  ptx::tmem_ld_32x32(tacc + c_lo, va);
#pragma unroll 1
  for (int c = c_lo; c < c_hi; c += 64) {
    ptx::tmem_ld_wait_for(va);
    const bool more = c + 32 < c_hi;
    if (more) ptx::tmem_ld_32x32(tacc + c + 32, vb);
    f(c, va);
    if (more) {
      ptx::tmem_ld_wait_for(vb);
      if (c + 64 < c_hi) ptx::tmem_ld_32x32(tacc + c + 64, va);
      f(c + 32, vb);
    }
  }
}

// Number of columns of [col_lo, col_hi) that lie below `limit` when the tile starts at global
// column `tile_col0`, rounded up to whole chunks: the exclusive end offset for for_each_chunk.
__device__ __forceinline__ int chunk_end(int tile_col0, int col_hi, int limit) {
  const int left = limit - tile_col0;
  if (left <= 0) return 0;
  const int up = (left + 31) & ~31;
  return up < col_hi ? up : col_hi;
}

__device__ __forceinline__ void store_bf16x32(uint16_t* dst, const float (&v)[32]) {
  uint4* out = reinterpret_cast<uint4*>(dst);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    uint4 w;
    w.x = ptx::pack_bf16x2(v[q * 8 + 0], v[q * 8 + 1]);
    w.y = ptx::pack_bf16x2(v[q * 8 + 2], v[q * 8 + 3]);
    w.z = ptx::pack_bf16x2(v[q * 8 + 4], v[q * 8 + 5]);
    w.w = ptx::pack_bf16x2(v[q * 8 + 6], v[q * 8 + 7]);
    out[q] = w;
  }
}

// bf16 output through shared memory and TMA: a warp owns one 4 KB slab = its 32 rows x 64 columns (128 bytes
// per row, 128-byte swizzle: the 16-byte piece q of row r sits at piece q ^ (r % 8), so the eight lanes
// that write together hit eight different bank groups).  Two 32-column chunks fill a slab; one lane then
// hands it to the TMA unit, which writes whole 128-byte lines and drops rows or columns beyond the
// tensor's extent.  Compared with every lane storing 16-byte pieces of its own row, the load/store pipe
// sees 16 instead of 128 wavefronts per chunk.
constexpr int kSlabBytes = 4096;

struct SlabStore {
  // `half` = which 32 columns of the slab; the first half first waits until the previous store of
  // this slab has been read out of shared memory.
  __device__ static __forceinline__ void put(uint8_t* block_smem, int epi_tid, const float (&v)[32], int half) {
    const int lane = epi_tid & 31;
    if (half == 0) {
      if (lane == 0) ptx::bulk_wait_group_read<0>();
      __syncwarp();
    }
    const uint32_t row = ptx::smem_u32(block_smem) + (epi_tid >> 5) * kSlabBytes + lane * 128;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint32_t addr = row + (((half * 4 + q) ^ (lane & 7)) << 4);
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr),
                   "r"(ptx::pack_bf16x2(v[q * 8 + 0], v[q * 8 + 1])), "r"(ptx::pack_bf16x2(v[q * 8 + 2], v[q * 8 + 3])),
                   "r"(ptx::pack_bf16x2(v[q * 8 + 4], v[q * 8 + 5])), "r"(ptx::pack_bf16x2(v[q * 8 + 6], v[q * 8 + 7]))
                   : "memory");
    }
  }
  // The slab is complete: write it to columns [col0, col0 + 64), rows [row0, row0 + 32) of the output.
  __device__ static __forceinline__ void flush(const CUtensorMap* out, uint8_t* block_smem, int epi_tid, int col0,
                                               int row0) {
    ptx::fence_proxy_async_smem();
    __syncwarp();
    if ((epi_tid & 31) == 0) {
      ptx::tma_store_2d(out, ptx::smem_u32(block_smem) + (epi_tid >> 5) * kSlabBytes, col0, row0);
      ptx::bulk_commit_group();
    }
  }
  // Before the thread leaves: its stores must have completed.
  __device__ static __forceinline__ void drain(int epi_tid) {
    if ((epi_tid & 31) == 0) ptx::bulk_wait_group_all();
  }
};

// acc += sum_j bf16(w)[j] * v[8*q + j] for the 8 bf16 values packed in w.
__device__ __forceinline__ float dot8(const uint4 w, const float* v, float acc) {
  acc = fmaf(ptx::bf16_lo(w.x), v[0], acc);
  acc = fmaf(ptx::bf16_hi(w.x), v[1], acc);
  acc = fmaf(ptx::bf16_lo(w.y), v[2], acc);
  acc = fmaf(ptx::bf16_hi(w.y), v[3], acc);
  acc = fmaf(ptx::bf16_lo(w.z), v[4], acc);
  acc = fmaf(ptx::bf16_hi(w.z), v[5], acc);
  acc = fmaf(ptx::bf16_lo(w.w), v[6], acc);
  acc = fmaf(ptx::bf16_hi(w.w), v[7], acc);
  return acc;
}
// v[j] += g * bf16(w)[j]
__device__ __forceinline__ void axpy8(const float g, const uint4 w, float* v) {
  v[0] = fmaf(g, ptx::bf16_lo(w.x), v[0]);
  v[1] = fmaf(g, ptx::bf16_hi(w.x), v[1]);
  v[2] = fmaf(g, ptx::bf16_lo(w.y), v[2]);
  v[3] = fmaf(g, ptx::bf16_hi(w.y), v[3]);
  v[4] = fmaf(g, ptx::bf16_lo(w.z), v[4]);
  v[5] = fmaf(g, ptx::bf16_hi(w.z), v[5]);
  v[6] = fmaf(g, ptx::bf16_lo(w.w), v[6]);
  v[7] = fmaf(g, ptx::bf16_hi(w.w), v[7]);
}

// ---------------------------------------------------------------------------
// Head projection (reduced head: W^(s)_alpha = W x w^(s)_alpha, applied to e_t).
//   z[i, k, :] = W_head[k] . h[i, :]  stored as bf16, one GEMM over all k.
// Side output: the target logit of Eq. 8 taken from the *unrounded* fp32 z,
//   tgt_part[i, (k*d + j0)/64] = sum_{j in 64-block} E[x[i, s(k)], j] * z[i, k, j],
// so that the bf16 rounding of z does not enter the target term.
// Requires d % 64 == 0 (a 64-column block never straddles two heads).
// The target token of every 64-column block is fetched before the accumulator is waited for, and the
// slice of E[x] that a chunk needs is fetched one chunk ahead, so neither load's latency sits between
// two chunks.
template <int BN>
struct EpiProj : EpiDefaults {
  struct Params {
    alignas(64) CUtensorMap z_map;   // z [M, ncols] bf16 as 64-column x 32-row boxes (the output of the TMA stores)
    uint16_t* z;            // [M, ncols] bf16
    float* tgt_part;        // [M, ncols / 64]
    const uint16_t* E;      // [V, d] bf16
    const int32_t* x;       // [M, n], or nullptr to skip the target-logit side output
    float* z32;             // [M, ncols] unrounded z for the draft sampler, or nullptr
    int* dev_status;
    int M, ncols, d, V, n, r;
  };
  struct State { int tok[BN / 64]; };
  static constexpr int SMEM_PER_WARP = kSlabBytes;
  __device__ static void unit_begin(const Params&, State&, int, int, int) {}
  __device__ static void unit_end(const Params&, State&, int, int, int, uint8_t*, int) {}
  __device__ static void role_end(const Params&, State&, uint8_t*, int epi_tid) { SlabStore::drain(epi_tid); }

  __device__ static void pre_tile(const Params& p, State& st, int m_tile, int n_tile, int row_in_tile) {
    const int row = m_tile * kBM + row_in_tile;
    if (p.x == nullptr || row >= p.M) return;
#pragma unroll
    for (int b = 0; b < BN / 64; ++b) {
      const int col0 = n_tile * BN + b * 64;
      if (col0 >= p.ncols) continue;
      const size_t xi = static_cast<size_t>(row) * p.n + (col0 / p.d) / p.r;
      int tok = CPMTP_INDEX_OK(xi, 1, static_cast<size_t>(p.M) * p.n) ? __ldg(p.x + xi) : 0;
      if (tok < 0 || tok >= p.V) {
        if (p.dev_status != nullptr) atomicMax(p.dev_status, kDevTargetOutOfRange);
        tok = tok < 0 ? 0 : p.V - 1;
      }
      st.tok[b] = tok;
    }
  }

  __device__ static void tile(const Params& p, State& st, uint32_t tacc, int m_tile, int n_tile, int row_in_tile,
                              uint8_t* smem, int epi_tid) {
    tile_part(p, st, tacc, m_tile, n_tile, row_in_tile, smem, epi_tid, 0, BN);
  }
  // Columns [c_begin, c_end) of the tile (multiples of 64): the whole tile, or the part of it that one of two
  // warps on the same accumulator rows handles.
  __device__ static void tile_part(const Params& p, State& st, uint32_t tacc, int m_tile, int n_tile, int row_in_tile,
                                   uint8_t* smem, int epi_tid, int c_begin, int c_end) {
    const int row = m_tile * kBM + row_in_tile;
    const bool valid = row < p.M;
    const bool gather = valid && p.x != nullptr;
    const int tile_col0 = n_tile * BN;
    const int c_hi = chunk_end(tile_col0, c_end, p.ncols);
    if (c_hi <= c_begin) return;
    // slice of the target row of E that chunk c multiplies: 32 bf16 = four 16-byte loads
    auto fetch = [&](int c, uint4 (&e)[4]) {
      if (!gather) return;
      const int col0 = tile_col0 + c;
      const int j0 = col0 % p.d;
      int tok = 0;
#pragma unroll
      for (int b = 0; b < BN / 64; ++b)
        if (b == (c >> 6)) tok = st.tok[b];
      const size_t ei = static_cast<size_t>(tok) * p.d + j0;
      const uint4* src = reinterpret_cast<const uint4*>(p.E + ei);
      const bool ok = CPMTP_INDEX_OK(ei, 32, static_cast<size_t>(p.V) * p.d);
#pragma unroll
      for (int q = 0; q < 4; ++q) e[q] = ok ? __ldg(src + q) : make_uint4(0u, 0u, 0u, 0u);
    };
    float part = 0.f;
    auto work = [&](int c, float (&v)[32], const uint4 (&e)[4]) {
      const int col0 = tile_col0 + c;
      // z as bf16: every lane takes part (rows beyond M are dropped by the store itself)
      SlabStore::put(smem, epi_tid, v, (c >> 5) & 1);
      if (c & 32) SlabStore::flush(&p.z_map, smem, epi_tid, col0 - 32, m_tile * kBM + (row_in_tile & ~31));
      if (!valid) return;
      if (p.z32 != nullptr &&
          CPMTP_INDEX_OK(static_cast<size_t>(row) * p.ncols + col0, 32, static_cast<size_t>(p.M) * p.ncols)) {
        float4* dst = reinterpret_cast<float4*>(p.z32 + static_cast<size_t>(row) * p.ncols + col0);
#pragma unroll
        for (int q = 0; q < 8; ++q) dst[q] = make_float4(v[q * 4], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3]);
      }
      if (!gather) return;
      float acc = 0.f;
#pragma unroll
      for (int q = 0; q < 4; ++q) acc = dot8(e[q], v + q * 8, acc);
      if ((c & 32) == 0) {
        part = acc;
      } else {
        const size_t ti = static_cast<size_t>(row) * (p.ncols >> 6) + (col0 >> 6);
        if (CPMTP_INDEX_OK(ti, 1, static_cast<size_t>(p.M) * (p.ncols >> 6))) p.tgt_part[ti] = part + acc;
      }
    };
    float va[32], vb[32];
    uint4 ea[4], eb[4];
    ptx::tmem_ld_32x32(tacc + c_begin, va);
    fetch(c_begin, ea);
#pragma unroll 1
    for (int c = c_begin; c < c_hi; c += 64) {
      ptx::tmem_ld_wait_for(va);
      const bool more = c + 32 < c_hi;   // always true here (ncols % 64 == 0); kept for symmetry
      if (more) {
        ptx::tmem_ld_32x32(tacc + c + 32, vb);
        fetch(c + 32, eb);
      }
      work(c, va, ea);
      if (more) {
        ptx::tmem_ld_wait_for(vb);
        if (c + 64 < c_hi) {
          ptx::tmem_ld_32x32(tacc + c + 64, va);
          fetch(c + 64, ea);
        }
        work(c + 32, vb, eb);
      }
    }
  }
};

// ---------------------------------------------------------------------------
// Unembedding fused with the vocabulary log-sum-exp of Eq. 5 / Eq. 8:
//   S[(i,k), v] = E[v, :] . z[i, k, :] never leaves TMEM/registers; each thread
// keeps a running (max, sum-exp) over the column tiles of its unit and writes
// one partial per (row, part).  Values are kept in the log2 domain.
// STORE = true additionally writes the raw logits (fp32) for the draft sampler, which needs
// whole distributions; the likelihood path never does.
__device__ __forceinline__ void online_lse_chunk(float (&v)[32], float& m2, float& l) {
  float cm = v[0];
#pragma unroll
  for (int j = 1; j < 32; ++j) cm = fmaxf(cm, v[j]);
  const float m_new = fmaxf(m2, cm * kLog2e);
  float sum = 0.f;
#pragma unroll
  for (int j = 0; j < 32; ++j) sum += ptx::ex2_approx(fmaf(v[j], kLog2e, -m_new));
  l = l * ptx::ex2_approx(m2 - m_new) + sum;
  m2 = m_new;
}

template <int BN, bool STORE = false>
struct EpiLse : EpiDefaults {
  struct Params {
    float* part_m;   // [M, parts] running max * log2(e)
    float* part_l;   // [M, parts] sum 2^(s*log2e - max)
    int M, V, parts;
    float* S;        // [M, lds] logits (STORE only); lds % 32 == 0, lds >= V
    int lds;
  };
  struct State { float m2, l; };
  __device__ static void unit_begin(const Params&, State& st, int, int, int) {
    st.m2 = -INFINITY;
    st.l = 0.f;
  }
  __device__ static void unit_end(const Params& p, State& st, int m_tile, int part, int row_in_tile,
                                  uint8_t*, int) {
    const int row = m_tile * kBM + row_in_tile;
    const size_t pi = static_cast<size_t>(row) * p.parts + part;
    if (row < p.M && CPMTP_INDEX_OK(pi, 1, static_cast<size_t>(p.M) * p.parts)) {
      p.part_m[pi] = st.m2;
      p.part_l[pi] = st.l;
    }
  }
  __device__ static void tile(const Params& p, State& st, uint32_t tacc, int m_tile, int n_tile,
                              int row_in_tile, uint8_t*, int) {
    const int tile_col0 = n_tile * BN;
    const int row = m_tile * kBM + row_in_tile;
    for_each_chunk(tacc, 0, chunk_end(tile_col0, BN, p.V), [&](int c, float (&v)[32]) {
      const int col0 = tile_col0 + c;
      if constexpr (STORE) {
        if (row < p.M &&
            CPMTP_INDEX_OK(static_cast<size_t>(row) * p.lds + col0, 32, static_cast<size_t>(p.M) * p.lds)) {
          float4* dst = reinterpret_cast<float4*>(p.S + static_cast<size_t>(row) * p.lds + col0);
#pragma unroll
          for (int q = 0; q < 8; ++q) dst[q] = make_float4(v[q * 4], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3]);
        }
      }
      if (col0 + 32 > p.V) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (col0 + j >= p.V) v[j] = -INFINITY;
      }
      online_lse_chunk(v, st.m2, st.l);
    });
  }
};

// ---------------------------------------------------------------------------
// Full head (Eq. 6 as printed: one unembedding per (token, expert)): the logits of all heads come
// from ONE GEMM  S[i, k*V + v] = W_full[k][v, :] . h[i, :]  whose column tiles are segmented by head.
// A unit stays inside one head; each thread keeps the running (max, sum-exp) of its row for that
// head, and picks the target logit straight from the fp32 accumulator when its column comes by.
template <int BN>
struct EpiLseFull : EpiDefaults {
  struct Params {
    float* part_m;       // [M, parts]  (parts = K * splits per head * column halves)
    float* part_l;
    float* tgt;          // [M, K]
    const int32_t* x;    // [M, n]
    int* dev_status;
    int M, V, K, n, r, tph, parts;   // tph = column tiles per head
  };
  struct State { float m2, l, tgt; int k, tok; };
  __device__ static void unit_begin(const Params&, State& st, int, int, int) {
    st.m2 = -INFINITY;
    st.l = 0.f;
    st.tgt = 0.f;
    st.k = -1;
    st.tok = -1;
  }
  __device__ static void unit_end(const Params& p, State& st, int m_tile, int part, int row_in_tile, uint8_t*, int) {
    const int row = m_tile * kBM + row_in_tile;
    const size_t pi = static_cast<size_t>(row) * p.parts + part;
    if (row < p.M && st.k >= 0 && CPMTP_INDEX_OK(pi, 1, static_cast<size_t>(p.M) * p.parts)) {
      p.part_m[pi] = st.m2;
      p.part_l[pi] = st.l;
      const size_t ti = static_cast<size_t>(row) * p.K + st.k;
      if (st.tok == -2 && CPMTP_INDEX_OK(ti, 1, static_cast<size_t>(p.M) * p.K)) p.tgt[ti] = st.tgt;   // these columns held the target
    }
  }
  __device__ static void tile(const Params& p, State& st, uint32_t tacc, int m_tile, int n_tile, int row_in_tile,
                              uint8_t*, int) {
    const int row = m_tile * kBM + row_in_tile;
    const int k = n_tile / p.tph;
    const int local0 = (n_tile - k * p.tph) * BN;
    if (st.k != k) {   // first tile of the unit (units never straddle heads)
      st.k = k;
      if (row < p.M) {
        const size_t xi = static_cast<size_t>(row) * p.n + k / p.r;
        int tok = CPMTP_INDEX_OK(xi, 1, static_cast<size_t>(p.M) * p.n) ? p.x[xi] : 0;
        if (tok < 0 || tok >= p.V) {
          if (p.dev_status != nullptr) atomicMax(p.dev_status, kDevTargetOutOfRange);
          tok = tok < 0 ? 0 : p.V - 1;
        }
        st.tok = tok;
      }
    }
    for_each_chunk(tacc, 0, chunk_end(local0, BN, p.V), [&](int c, float (&v)[32]) {
      const int col0 = local0 + c;
      const int t = st.tok - col0;
      if (t >= 0 && t < 32) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (j == t) st.tgt = v[j];
        st.tok = -2;
      }
      if (col0 + 32 > p.V) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (col0 + j >= p.V) v[j] = -INFINITY;
      }
      online_lse_chunk(v, st.m2, st.l);
    });
  }
};

// ---------------------------------------------------------------------------
// Backward: recompute a logits tile and turn it into the logit gradient
//   G[(i,k), v] = c[i, alpha(k)] * (1[v = x[i, s(k)]] - exp(S - lse[i,k]))
// (derivative of Eq. 9 through Eq. 8), stored as bf16 for the two GEMMs that
// consume it.  Rows are relative to a chunk starting at global row `row0`.
// Columns in [V, ldg) are written as zero; ldg % 32 == 0.
__device__ __forceinline__ void logit_grad_chunk(float (&v)[32], int col0, int V, int tok, float lse2, float coef) {
  const float nc = -coef;
#pragma unroll
  for (int j = 0; j < 32; ++j) v[j] = nc * ptx::ex2_approx(fmaf(v[j], kLog2e, -lse2));
  const int t = tok - col0;
  if (t >= 0 && t < 32) {
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (j == t) v[j] += coef;
  }
  if (col0 + 32 > V) {
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (col0 + j >= V) v[j] = 0.f;
  }
}

template <int BN>
struct EpiLogitGrad : EpiDefaults {
  struct Params {
    alignas(64) CUtensorMap G_map;   // G [rows, ldg] bf16 as 64-column x 32-row boxes
    uint16_t* G;          // [rows, ldg] bf16
    const float* lse;     // [N*K]
    const float* coef;    // [N, K]  d objective / d C per head
    const int32_t* x;     // [N, n]
    long long row0;
    int rows, ldg, V, K, n, r;
  };
  struct State { float lse2, coef; int tok; };
  static constexpr int SMEM_PER_WARP = kSlabBytes;
  __device__ static void role_end(const Params&, State&, uint8_t*, int epi_tid) { SlabStore::drain(epi_tid); }
  __device__ static void unit_begin(const Params& p, State& st, int m_tile, int, int row_in_tile) {
    const int row = m_tile * kBM + row_in_tile;
    st.lse2 = 0.f;
    st.coef = 0.f;
    st.tok = -1;
    if (row < p.rows) {
      const long long grow = p.row0 + row;
      const long long i = grow / p.K;
      const int k = static_cast<int>(grow - i * p.K);
      st.lse2 = p.lse[grow] * kLog2e;
      st.coef = p.coef[grow];
      const long long xi = i * p.n + k / p.r;
      const int tok = CPMTP_INDEX_OK(xi, 1, (p.row0 + p.rows + p.K - 1) / p.K * p.n) ? p.x[xi] : 0;
      st.tok = tok < 0 ? 0 : (tok >= p.V ? p.V - 1 : tok);
    }
  }
  __device__ static void unit_end(const Params&, State&, int, int, int, uint8_t*, int) {}
  __device__ static void tile(const Params& p, State& st, uint32_t tacc, int m_tile, int n_tile,
                              int row_in_tile, uint8_t* smem, int epi_tid) {
    const int tile_col0 = n_tile * BN;
    // ldg % 64 == 0: the columns below ldg form whole 64-column slabs
    for_each_chunk(tacc, 0, chunk_end(tile_col0, BN, p.ldg), [&](int c, float (&v)[32]) {
      const int col0 = tile_col0 + c;
      logit_grad_chunk(v, col0, p.V, st.tok, st.lse2, st.coef);
      SlabStore::put(smem, epi_tid, v, (c >> 5) & 1);
      if (c & 32) SlabStore::flush(&p.G_map, smem, epi_tid, col0 - 32, m_tile * kBM + (row_in_tile & ~31));
    });
  }
};

// ---------------------------------------------------------------------------
// Full head, backward: the logit gradient of a few heads [k0, k0 + heads) at a time,
//   G[i, (k - k0) * ldv + v] = c[i, alpha(k)] * (1[v = x[i, s(k)]] - exp(S[i,k,v] - lse[i,k])),
// from the same segmented GEMM as the forward.  Columns in [V, ldv) of every head are zero.
template <int BN>
struct EpiLogitGradFull : EpiDefaults {
  struct Params {
    alignas(64) CUtensorMap G_map;   // G [M, ldg] bf16 as 64-column x 32-row boxes
    uint16_t* G;          // [M, ldg] bf16, ldg = heads * ldv
    const float* lse;     // [M, K]
    const float* coef;    // [M, K]  d objective / d C per head
    const int32_t* x;     // [M, n]
    int M, V, K, n, r, tph, ldv, ldg, k0;
  };
  struct State { float lse2, coef; int tok, k; };
  static constexpr int SMEM_PER_WARP = kSlabBytes;
  __device__ static void role_end(const Params&, State&, uint8_t*, int epi_tid) { SlabStore::drain(epi_tid); }
  __device__ static void unit_begin(const Params&, State& st, int, int, int) { st.k = -1; }
  __device__ static void unit_end(const Params&, State&, int, int, int, uint8_t*, int) {}
  __device__ static void tile(const Params& p, State& st, uint32_t tacc, int m_tile, int n_tile, int row_in_tile,
                              uint8_t* smem, int epi_tid) {
    const int row = m_tile * kBM + row_in_tile;
    const bool valid = row < p.M;
    const int k_local = n_tile / p.tph;
    const int local0 = (n_tile - k_local * p.tph) * BN;
    const int k = p.k0 + k_local;
    if (st.k != k) {
      st.k = k;
      st.lse2 = 0.f;
      st.coef = 0.f;
      st.tok = -1;
      if (valid) {
        st.lse2 = p.lse[static_cast<size_t>(row) * p.K + k] * kLog2e;
        st.coef = p.coef[static_cast<size_t>(row) * p.K + k];
        const size_t xi = static_cast<size_t>(row) * p.n + k / p.r;
        const int tok = CPMTP_INDEX_OK(xi, 1, static_cast<size_t>(p.M) * p.n) ? p.x[xi] : 0;
        st.tok = tok < 0 ? 0 : (tok >= p.V ? p.V - 1 : tok);
      }
    }
    for_each_chunk(tacc, 0, chunk_end(local0, BN, p.ldv), [&](int c, float (&v)[32]) {
      const int col0 = local0 + c;
      logit_grad_chunk(v, col0, p.V, st.tok, st.lse2, st.coef);
      SlabStore::put(smem, epi_tid, v, (c >> 5) & 1);
      if (c & 32) SlabStore::flush(&p.G_map, smem, epi_tid, k_local * p.ldv + col0 - 32, m_tile * kBM + (row_in_tile & ~31));
    });
  }
};

// v[j] += bf16 values already stored at dst[0..32)
__device__ __forceinline__ void add_bf16x32(const uint16_t* dst, float (&v)[32]) {
  const uint4* in = reinterpret_cast<const uint4*>(dst);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint4 w = in[q];
    v[q * 8 + 0] += ptx::bf16_lo(w.x); v[q * 8 + 1] += ptx::bf16_hi(w.x);
    v[q * 8 + 2] += ptx::bf16_lo(w.y); v[q * 8 + 3] += ptx::bf16_hi(w.y);
    v[q * 8 + 4] += ptx::bf16_lo(w.z); v[q * 8 + 5] += ptx::bf16_hi(w.z);
    v[q * 8 + 6] += ptx::bf16_lo(w.w); v[q * 8 + 7] += ptx::bf16_hi(w.w);
  }
}

// ---------------------------------------------------------------------------
// Plain bf16 store, optionally adding the gate path  sum_beta dg[row, beta] * W_g[beta, col]
// (used for dh, where the gate logits of Eq. 7 contribute W_g^T dg).  With `accumulate` the
// value already in C is added before rounding (gradient accumulation over micro-batches).
// ncols must be a multiple of 32.
template <int BN, bool GATE>
struct EpiStoreBf16 : EpiDefaults {
  struct Params {
    uint16_t* C;           // [M, ldc] bf16
    const float* dg;       // [M, r]      (GATE only)
    const uint16_t* W_g;   // [r, ncols]  (GATE only)
    int M, ncols, ldc, r;
    int accumulate;        // C += result instead of C = result
  };
  struct State {};
  __device__ static void unit_begin(const Params&, State&, int, int, int) {}
  __device__ static void unit_end(const Params&, State&, int, int, int, uint8_t*, int) {}
  __device__ static void tile(const Params& p, State&, uint32_t tacc, int m_tile, int n_tile,
                              int row_in_tile, uint8_t*, int) {
    const int row = m_tile * kBM + row_in_tile;
    const bool valid = row < p.M;
    const int tile_col0 = n_tile * BN;
    for_each_chunk(tacc, 0, chunk_end(tile_col0, BN, p.ncols), [&](int c, float (&v)[32]) {
      if (!valid) return;
      const int col0 = tile_col0 + c;
      if constexpr (GATE) {
        for (int b = 0; b < p.r; ++b) {
          if (!CPMTP_INDEX_OK(static_cast<size_t>(b) * p.ncols + col0, 32, static_cast<size_t>(p.r) * p.ncols)) continue;
          const float g = p.dg[static_cast<size_t>(row) * p.r + b];
          const uint4* w = reinterpret_cast<const uint4*>(p.W_g + static_cast<size_t>(b) * p.ncols + col0);
#pragma unroll
          for (int q = 0; q < 4; ++q) axpy8(g, __ldg(w + q), v + q * 8);
        }
      }
      const size_t ci = static_cast<size_t>(row) * p.ldc + col0;
      if (!CPMTP_INDEX_OK(ci, 32, static_cast<size_t>(p.M - 1) * p.ldc + p.ncols)) return;
      uint16_t* dst = p.C + ci;
      if (p.accumulate) add_bf16x32(dst, v);
      store_bf16x32(dst, v);
    });
  }
};

// ---------------------------------------------------------------------------
// fp32 store / accumulate (dE summed over row chunks).  ncols multiple of 32.
template <int BN>
struct EpiAccumF32 : EpiDefaults {
  struct Params {
    float* C;   // [M, ldc]
    int M, ncols, ldc, accumulate;
  };
  struct State {};
  __device__ static void unit_begin(const Params&, State&, int, int, int) {}
  __device__ static void unit_end(const Params&, State&, int, int, int, uint8_t*, int) {}
  __device__ static void tile(const Params& p, State&, uint32_t tacc, int m_tile, int n_tile,
                              int row_in_tile, uint8_t*, int) {
    const int row = m_tile * kBM + row_in_tile;
    const bool valid = row < p.M;
    const int tile_col0 = n_tile * BN;
    for_each_chunk(tacc, 0, chunk_end(tile_col0, BN, p.ncols), [&](int c, float (&v)[32]) {
      if (!valid) return;
      const size_t ci = static_cast<size_t>(row) * p.ldc + tile_col0 + c;
      if (!CPMTP_INDEX_OK(ci, 32, static_cast<size_t>(p.M - 1) * p.ldc + p.ncols)) return;
      float4* dst = reinterpret_cast<float4*>(p.C + ci);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        float4 o = make_float4(v[q * 4 + 0], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3]);
        if (p.accumulate) {
          const float4 old = dst[q];
          o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
        }
        dst[q] = o;
      }
    });
  }
};

}  // namespace cpmtp
