// Epilogues plugged into the tcgen05 GEMM engine.  Each one consumes a
// 128 x BN fp32 accumulator tile straight from TMEM; thread `row_in_tile` owns
// one accumulator row and walks it in 32-column chunks.
#pragma once
#include <cstdint>

#include "ptx.cuh"
#include "tc_gemm.cuh"

namespace cpmtp {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

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
template <int BN>
struct EpiProj {
  struct Params {
    uint16_t* z;            // [M, ncols] bf16
    float* tgt_part;        // [M, ncols / 64]
    const uint16_t* E;      // [V, d] bf16
    const int32_t* x;       // [M, n], or nullptr to skip the target-logit side output
    float* z32;             // [M, ncols] unrounded z for the draft sampler, or nullptr
    int* dev_status;
    int M, ncols, d, V, n, r;
  };
  struct State {};
  static constexpr int SMEM_BYTES = 0;
  __device__ static void unit_begin(const Params&, State&, int, int, int) {}
  __device__ static void unit_end(const Params&, State&, int, int, int, uint8_t*, int) {}

  __device__ static void tile(const Params& p, State&, uint32_t tacc, int m_tile, int n_tile,
                              int row_in_tile, uint8_t*, int) {
    const int row = m_tile * kBM + row_in_tile;
    const bool valid = row < p.M;
    float part = 0.f;
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
      const int col0 = n_tile * BN + c;
      if (col0 >= p.ncols) break;   // uniform
      float v[32];
      ptx::tmem_ld_32x32(tacc + c, v);
      ptx::tmem_ld_wait();
      if (valid) {
        store_bf16x32(p.z + static_cast<size_t>(row) * p.ncols + col0, v);
        if (p.z32 != nullptr) {
          float4* dst = reinterpret_cast<float4*>(p.z32 + static_cast<size_t>(row) * p.ncols + col0);
#pragma unroll
          for (int q = 0; q < 8; ++q) dst[q] = make_float4(v[q * 4], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3]);
        }
        if (p.x == nullptr) continue;   // no targets (draft generation): only z is needed
        const int k = col0 / p.d;
        const int j0 = col0 - k * p.d;
        int tok = p.x[static_cast<size_t>(row) * p.n + k / p.r];
        if (tok < 0 || tok >= p.V) {
          if (p.dev_status != nullptr) atomicMax(p.dev_status, kDevTargetOutOfRange);
          tok = tok < 0 ? 0 : p.V - 1;
        }
        const uint4* e = reinterpret_cast<const uint4*>(p.E + static_cast<size_t>(tok) * p.d + j0);
        float acc = 0.f;
#pragma unroll
        for (int q = 0; q < 4; ++q) acc = dot8(__ldg(e + q), v + q * 8, acc);
        if ((c & 32) == 0) {
          part = acc;
        } else {
          p.tgt_part[static_cast<size_t>(row) * (p.ncols >> 6) + (col0 >> 6)] = part + acc;
        }
      }
    }
  }
};

// ---------------------------------------------------------------------------
// Unembedding fused with the vocabulary log-sum-exp of Eq. 5 / Eq. 8:
//   S[(i,k), v] = E[v, :] . z[i, k, :] never leaves TMEM/registers; each thread
// keeps a running (max, sum-exp) over the column tiles of its unit and writes
// one partial per (row, split).  Values are kept in the log2 domain.
// STORE = true additionally writes the raw logits (fp32) for the draft sampler, which needs
// whole distributions; the likelihood path never does.
template <int BN, bool STORE = false>
struct EpiLse {
  struct Params {
    float* part_m;   // [M, splits] running max * log2(e)
    float* part_l;   // [M, splits] sum 2^(s*log2e - max)
    int M, V, splits;
    float* S;        // [M, lds] logits (STORE only); lds % 32 == 0, lds >= V
    int lds;
  };
  struct State { float m2, l; };
  static constexpr int SMEM_BYTES = 0;
  __device__ static void unit_begin(const Params&, State& st, int, int, int) {
    st.m2 = -INFINITY;
    st.l = 0.f;
  }
  __device__ static void unit_end(const Params& p, State& st, int m_tile, int split, int row_in_tile,
                                  uint8_t*, int) {
    const int row = m_tile * kBM + row_in_tile;
    if (row < p.M) {
      p.part_m[static_cast<size_t>(row) * p.splits + split] = st.m2;
      p.part_l[static_cast<size_t>(row) * p.splits + split] = st.l;
    }
  }
  __device__ static void tile(const Params& p, State& st, uint32_t tacc, int m_tile, int n_tile,
                              int row_in_tile, uint8_t*, int) {
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
      const int col0 = n_tile * BN + c;
      if (col0 >= p.V) break;   // uniform across the CTA
      float v[32];
      ptx::tmem_ld_32x32(tacc + c, v);
      ptx::tmem_ld_wait();
      if constexpr (STORE) {
        const int row = m_tile * kBM + row_in_tile;
        if (row < p.M) {
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
      float cm = v[0];
#pragma unroll
      for (int j = 1; j < 32; ++j) cm = fmaxf(cm, v[j]);
      const float m_new = fmaxf(st.m2, cm * kLog2e);
      float sum = 0.f;
#pragma unroll
      for (int j = 0; j < 32; ++j) sum += ptx::ex2_approx(fmaf(v[j], kLog2e, -m_new));
      st.l = st.l * ptx::ex2_approx(st.m2 - m_new) + sum;
      st.m2 = m_new;
    }
  }
};

// ---------------------------------------------------------------------------
// Full head (Eq. 6 as printed: one unembedding per (token, expert)): the logits of all heads come
// from ONE GEMM  S[i, k*V + v] = W_full[k][v, :] . h[i, :]  whose column tiles are segmented by head.
// A unit stays inside one head; each thread keeps the running (max, sum-exp) of its row for that
// head, and picks the target logit straight from the fp32 accumulator when its column comes by.
template <int BN>
struct EpiLseFull {
  struct Params {
    float* part_m;       // [M, K * sph]  (sph = splits per head)
    float* part_l;
    float* tgt;          // [M, K]
    const int32_t* x;    // [M, n]
    int* dev_status;
    int M, V, K, n, r, tph, n_splits;   // tph = column tiles per head
  };
  struct State { float m2, l, tgt; int k, tok; };
  static constexpr int SMEM_BYTES = 0;
  __device__ static void unit_begin(const Params&, State& st, int, int, int) {
    st.m2 = -INFINITY;
    st.l = 0.f;
    st.tgt = 0.f;
    st.k = -1;
    st.tok = -1;
  }
  __device__ static void unit_end(const Params& p, State& st, int m_tile, int split, int row_in_tile, uint8_t*, int) {
    const int row = m_tile * kBM + row_in_tile;
    if (row < p.M && st.k >= 0) {
      p.part_m[static_cast<size_t>(row) * p.n_splits + split] = st.m2;
      p.part_l[static_cast<size_t>(row) * p.n_splits + split] = st.l;
      if (st.tok == -2) p.tgt[static_cast<size_t>(row) * p.K + st.k] = st.tgt;   // this unit held the target column
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
        int tok = p.x[static_cast<size_t>(row) * p.n + k / p.r];
        if (tok < 0 || tok >= p.V) {
          if (p.dev_status != nullptr) atomicMax(p.dev_status, kDevTargetOutOfRange);
          tok = tok < 0 ? 0 : p.V - 1;
        }
        st.tok = tok;
      }
    }
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
      const int col0 = local0 + c;
      if (col0 >= p.V) break;   // uniform across the CTA
      float v[32];
      ptx::tmem_ld_32x32(tacc + c, v);
      ptx::tmem_ld_wait();
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
      float cm = v[0];
#pragma unroll
      for (int j = 1; j < 32; ++j) cm = fmaxf(cm, v[j]);
      const float m_new = fmaxf(st.m2, cm * kLog2e);
      float sum = 0.f;
#pragma unroll
      for (int j = 0; j < 32; ++j) sum += ptx::ex2_approx(fmaf(v[j], kLog2e, -m_new));
      st.l = st.l * ptx::ex2_approx(st.m2 - m_new) + sum;
      st.m2 = m_new;
    }
  }
};

// ---------------------------------------------------------------------------
// Backward: recompute a logits tile and turn it into the logit gradient
//   G[(i,k), v] = c[i, alpha(k)] * (1[v = x[i, s(k)]] - exp(S - lse[i,k]))
// (derivative of Eq. 9 through Eq. 8), stored as bf16 for the two GEMMs that
// consume it.  Rows are relative to a chunk starting at global row `row0`.
// Columns in [V, ldg) are written as zero; ldg % 32 == 0.
template <int BN>
struct EpiLogitGrad {
  struct Params {
    uint16_t* G;          // [rows, ldg] bf16
    const float* lse;     // [N*K]
    const float* coef;    // [N, K]  d objective / d C per head
    const int32_t* x;     // [N, n]
    long long row0;
    int rows, ldg, V, K, n, r;
  };
  struct State { float lse2, coef; int tok; };
  static constexpr int SMEM_BYTES = 0;
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
      const int tok = p.x[i * p.n + k / p.r];
      st.tok = tok < 0 ? 0 : (tok >= p.V ? p.V - 1 : tok);
    }
  }
  __device__ static void unit_end(const Params&, State&, int, int, int, uint8_t*, int) {}
  __device__ static void tile(const Params& p, State& st, uint32_t tacc, int m_tile, int n_tile,
                              int row_in_tile, uint8_t*, int) {
    const int row = m_tile * kBM + row_in_tile;
    const bool valid = row < p.rows;
    const float nc = -st.coef;
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
      const int col0 = n_tile * BN + c;
      if (col0 >= p.ldg) break;
      float v[32];
      ptx::tmem_ld_32x32(tacc + c, v);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = nc * ptx::ex2_approx(fmaf(v[j], kLog2e, -st.lse2));
      const int t = st.tok - col0;
      if (t >= 0 && t < 32) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (j == t) v[j] += st.coef;
      }
      if (col0 + 32 > p.V) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (col0 + j >= p.V) v[j] = 0.f;
      }
      if (valid) store_bf16x32(p.G + static_cast<size_t>(row) * p.ldg + col0, v);
    }
  }
};

// ---------------------------------------------------------------------------
// Full head, backward: the logit gradient of a few heads [k0, k0 + heads) at a time,
//   G[i, (k - k0) * ldv + v] = c[i, alpha(k)] * (1[v = x[i, s(k)]] - exp(S[i,k,v] - lse[i,k])),
// from the same segmented GEMM as the forward.  Columns in [V, ldv) of every head are zero.
template <int BN>
struct EpiLogitGradFull {
  struct Params {
    uint16_t* G;          // [M, ldg] bf16, ldg = heads * ldv
    const float* lse;     // [M, K]
    const float* coef;    // [M, K]  d objective / d C per head
    const int32_t* x;     // [M, n]
    int M, V, K, n, r, tph, ldv, ldg, k0;
  };
  struct State { float lse2, coef; int tok, k; };
  static constexpr int SMEM_BYTES = 0;
  __device__ static void unit_begin(const Params&, State& st, int, int, int) { st.k = -1; }
  __device__ static void unit_end(const Params&, State&, int, int, int, uint8_t*, int) {}
  __device__ static void tile(const Params& p, State& st, uint32_t tacc, int m_tile, int n_tile, int row_in_tile,
                              uint8_t*, int) {
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
        const int tok = p.x[static_cast<size_t>(row) * p.n + k / p.r];
        st.tok = tok < 0 ? 0 : (tok >= p.V ? p.V - 1 : tok);
      }
    }
    const float nc = -st.coef;
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
      const int col0 = local0 + c;
      if (col0 >= p.ldv) break;
      float v[32];
      ptx::tmem_ld_32x32(tacc + c, v);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = nc * ptx::ex2_approx(fmaf(v[j], kLog2e, -st.lse2));
      const int t = st.tok - col0;
      if (t >= 0 && t < 32) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (j == t) v[j] += st.coef;
      }
      if (col0 + 32 > p.V) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (col0 + j >= p.V) v[j] = 0.f;
      }
      if (valid) store_bf16x32(p.G + static_cast<size_t>(row) * p.ldg + static_cast<size_t>(k_local) * p.ldv + col0, v);
    }
  }
};

// ---------------------------------------------------------------------------
// Plain bf16 store, optionally adding the gate path  sum_beta dg[row, beta] * W_g[beta, col]
// (used for dh, where the gate logits of Eq. 7 contribute W_g^T dg).
// ncols must be a multiple of 32.
template <int BN, bool GATE>
struct EpiStoreBf16 {
  struct Params {
    uint16_t* C;           // [M, ldc] bf16
    const float* dg;       // [M, r]      (GATE only)
    const uint16_t* W_g;   // [r, ncols]  (GATE only)
    int M, ncols, ldc, r;
  };
  struct State {};
  static constexpr int SMEM_BYTES = 0;
  __device__ static void unit_begin(const Params&, State&, int, int, int) {}
  __device__ static void unit_end(const Params&, State&, int, int, int, uint8_t*, int) {}
  __device__ static void tile(const Params& p, State&, uint32_t tacc, int m_tile, int n_tile,
                              int row_in_tile, uint8_t*, int) {
    const int row = m_tile * kBM + row_in_tile;
    const bool valid = row < p.M;
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
      const int col0 = n_tile * BN + c;
      if (col0 >= p.ncols) break;
      float v[32];
      ptx::tmem_ld_32x32(tacc + c, v);
      ptx::tmem_ld_wait();
      if constexpr (GATE) {
        if (valid) {
          for (int b = 0; b < p.r; ++b) {
            const float g = p.dg[static_cast<size_t>(row) * p.r + b];
            const uint4* w = reinterpret_cast<const uint4*>(p.W_g + static_cast<size_t>(b) * p.ncols + col0);
#pragma unroll
            for (int q = 0; q < 4; ++q) axpy8(g, __ldg(w + q), v + q * 8);
          }
        }
      }
      if (valid) store_bf16x32(p.C + static_cast<size_t>(row) * p.ldc + col0, v);
    }
  }
};

// ---------------------------------------------------------------------------
// fp32 store / accumulate (dE summed over row chunks).  ncols multiple of 32.
template <int BN>
struct EpiAccumF32 {
  struct Params {
    float* C;   // [M, ldc]
    int M, ncols, ldc, accumulate;
  };
  struct State {};
  static constexpr int SMEM_BYTES = 0;
  __device__ static void unit_begin(const Params&, State&, int, int, int) {}
  __device__ static void unit_end(const Params&, State&, int, int, int, uint8_t*, int) {}
  __device__ static void tile(const Params& p, State&, uint32_t tacc, int m_tile, int n_tile,
                              int row_in_tile, uint8_t*, int) {
    const int row = m_tile * kBM + row_in_tile;
    const bool valid = row < p.M;
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
      const int col0 = n_tile * BN + c;
      if (col0 >= p.ncols) break;
      float v[32];
      ptx::tmem_ld_32x32(tacc + c, v);
      ptx::tmem_ld_wait();
      if (valid) {
        float4* dst = reinterpret_cast<float4*>(p.C + static_cast<size_t>(row) * p.ldc + col0);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          float4 o = make_float4(v[q * 4 + 0], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3]);
          if (p.accumulate) {
            const float4 old = dst[q];
            o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
          }
          dst[q] = o;
        }
      }
    }
  }
};

}  // namespace cpmtp
