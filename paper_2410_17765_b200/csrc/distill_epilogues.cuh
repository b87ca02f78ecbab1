// Epilogues of the distillation objective (Eq. 14): the KL term between the head's conditional
// next-token distribution p^d_k = sum_a pi_{k,a} P^(k)(. | a) and a frozen model's p^c_k.
//
// Both run on the unembedding GEMM with GROUPED rows: the r experts of one (position, token)
// pair sit in adjacent accumulator rows, padded to R = the next power of two (Sched::a_groups),
// so one group is R adjacent lanes of a warp and the mixture over experts is a lane exchange:
// a reduce-scatter leaves every lane with the full sum for 32 / R of the chunk's 32 columns, the
// lane finishes those columns (logarithm, teacher logit), and an all-gather hands the results back.
#pragma once
#include <cstdint>

#include "epilogues.cuh"

namespace cpmtp {

template <int R>
struct GroupLanes {
  static_assert(R == 1 || R == 2 || R == 4 || R == 8 || R == 16 || R == 32, "group size: a power of two <= 32");
  static constexpr int Q = R == 1 ? 0 : R == 2 ? 1 : R == 4 ? 2 : R == 8 ? 3 : R == 16 ? 4 : 5;
  static constexpr int W = 32 / R;   // columns a lane finishes per 32-column chunk

  // In: a[0..32) per lane.  Out: a[i], i < W, = sum over the group's lanes of their a[sub * W + i].
  __device__ static __forceinline__ void reduce_scatter(float (&a)[32], int sub) {
#pragma unroll
    for (int j = 0; j < Q; ++j) {
      const int half = 16 >> j;
      const int bit = Q - 1 - j;
      const bool up = (sub >> bit) & 1;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        if (i < half) {
          const float send = up ? a[i] : a[i + half];
          const float keep = up ? a[i + half] : a[i];
          a[i] = keep + __shfl_xor_sync(0xffffffffu, send, 1 << bit);
        }
      }
    }
  }
  // In: a[i], i < W, the values of columns sub * W + i.  Out: a[0..32) complete in every lane.
  __device__ static __forceinline__ void all_gather(float (&a)[32], int sub) {
#pragma unroll
    for (int j = Q - 1; j >= 0; --j) {
      const int half = 16 >> j;
      const int bit = Q - 1 - j;
      const bool up = (sub >> bit) & 1;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        if (i < half) {
          const float mine = a[i];
          const float other = __shfl_xor_sync(0xffffffffu, mine, 1 << bit);
          a[i + half] = up ? mine : other;
          a[i] = up ? other : mine;
        }
      }
    }
  }
};

// l(v) = log p^d(v) - log p^c(v) for the W columns [col, col + W) this lane finishes; pd[i] holds
// p^d on entry and l on exit.  Columns beyond V, rows beyond the last group and a p^d below the
// smallest normal float (every term underflowed; its weight in the sums is negligible too) give l = 0.
// vec: V % 8 == 0, so the teacher row is 16-byte aligned and pieces of <= 8 columns never straddle V.
// STATS: also fold the teacher logits read here into a running (max, sum-exp) in the log2 domain, so
// that the teacher's logsumexp needs no pass of its own.
template <int W, bool STATS = false>
__device__ __forceinline__ void finish_columns(float* pd, const uint16_t* __restrict__ trow, int col, int V,
                                               bool row_ok, bool vec, float lse_t, float* tm2 = nullptr,
                                               float* tl = nullptr) {
  constexpr int P = W < 8 ? W : 8;
#pragma unroll
  for (int q = 0; q < W / P; ++q) {
    const int c = col + q * P;
    float t[P];
#pragma unroll
    for (int i = 0; i < P; ++i) t[i] = 0.f;
    if (row_ok && c < V && CPMTP_INDEX_OK(c, vec ? P : 1, V)) {
      if (vec) {
        if constexpr (P == 8) {
          const uint4 u = __ldg(reinterpret_cast<const uint4*>(trow + c));
          t[0] = ptx::bf16_lo(u.x); t[1] = ptx::bf16_hi(u.x); t[2] = ptx::bf16_lo(u.y); t[3] = ptx::bf16_hi(u.y);
          t[4] = ptx::bf16_lo(u.z); t[5] = ptx::bf16_hi(u.z); t[6] = ptx::bf16_lo(u.w); t[7] = ptx::bf16_hi(u.w);
        } else if constexpr (P == 4) {
          const uint2 u = __ldg(reinterpret_cast<const uint2*>(trow + c));
          t[0] = ptx::bf16_lo(u.x); t[1] = ptx::bf16_hi(u.x); t[2] = ptx::bf16_lo(u.y); t[3] = ptx::bf16_hi(u.y);
        } else if constexpr (P == 2) {
          const uint32_t u = __ldg(reinterpret_cast<const uint32_t*>(trow + c));
          t[0] = ptx::bf16_lo(u); t[1] = ptx::bf16_hi(u);
        } else {
          t[0] = __uint_as_float(static_cast<uint32_t>(__ldg(trow + c)) << 16);
        }
      } else {
#pragma unroll
        for (int i = 0; i < P; ++i)
          if (c + i < V) t[i] = __uint_as_float(static_cast<uint32_t>(__ldg(trow + c + i)) << 16);
      }
    }
    if constexpr (STATS) {
      if (row_ok && c < V) {
        float cm = -INFINITY;
#pragma unroll
        for (int i = 0; i < P; ++i)
          if (c + i < V) cm = fmaxf(cm, t[i]);
        const float m_new = fmaxf(*tm2, cm * kLog2e);
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < P; ++i)
          if (c + i < V) sum += ptx::ex2_approx(fmaf(t[i], kLog2e, -m_new));
        *tl = *tl * ptx::ex2_approx(*tm2 - m_new) + sum;
        *tm2 = m_new;
      }
    }
#pragma unroll
    for (int i = 0; i < P; ++i) {
      const float p = pd[q * P + i];
      const bool ok = row_ok && (c + i < V) && p >= 1.17549435e-38f;   // lg2.approx flushes subnormals to -inf
      pd[q * P + i] = ok ? fmaf(ptx::lg2_approx(p), kLn2, lse_t - t[i]) : 0.f;
    }
  }
}

// ---------------------------------------------------------------------------
// Forward: pm[(g, a)] = sum_v e(v) l(v) with e = pi_{g,a} P^(k)(v | a); the KL term of Eq. 14 for
// group g is sum_a pm[(g, a)].  One partial per (row, split); rows are ORIGINAL rows g * r + a.
// The teacher's normaliser logsumexp_v T is not known during the sweep; it enters l(v) as a constant, and
// sum_v e(v) = pi, so the sweep accumulates  pm' = sum_v e(v) (log p^d(v) - T(v))  together with the running
// (max, sum-exp) of the teacher logits it reads anyway, and the merge kernel finishes  pm = pm' + pi * lse_t.
// Every teacher element is therefore read exactly once.
struct KlParams {
  float* part;            // [groups * r, splits]  pm' partials
  float* part_tm;         // [groups, splits]      running max of T * log2(e)
  float* part_tl;         // [groups, splits]      sum 2^(T * log2(e) - max)
  const float* lse;       // [groups * r]  logsumexp_v S
  const float* logpi;     // [groups * r]  log pi
  const uint16_t* T;      // [groups, V]   teacher logits, bf16
  int groups, r, V, splits, vec;
};

template <int BN, int R>
struct EpiKl : EpiDefaults {
  using Params = KlParams;
  struct State { float c2, tm2, tl, acc; long long orow; int grp; bool valid, grp_ok; };
  using GL = GroupLanes<R>;
  __device__ static void unit_begin(const Params& p, State& st, int m_tile, int, int row_in_tile) {
    st.grp = m_tile * (kBM / R) + row_in_tile / R;
    const int a = row_in_tile % R;
    st.grp_ok = st.grp < p.groups;
    st.valid = st.grp_ok && a < p.r;
    st.orow = static_cast<long long>(st.grp) * p.r + a;
    st.c2 = st.valid ? (p.logpi[st.orow] - p.lse[st.orow]) * kLog2e : -INFINITY;
    st.tm2 = -INFINITY;
    st.tl = 0.f;
    st.acc = 0.f;
  }
  __device__ static void unit_end(const Params& p, State& st, int, int split, int row_in_tile, uint8_t*, int) {
    const size_t pi = static_cast<size_t>(st.orow) * p.splits + split;
    if (st.valid && CPMTP_INDEX_OK(pi, 1, static_cast<size_t>(p.groups) * p.r * p.splits)) p.part[pi] = st.acc;
    // teacher statistics: every lane of the group holds those of its own columns; combine over the group
    float m = st.tm2;
#pragma unroll
    for (int o = R >> 1; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float l = st.tl > 0.f ? st.tl * ptx::ex2_approx(st.tm2 - m) : 0.f;
#pragma unroll
    for (int o = R >> 1; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    const size_t ti = static_cast<size_t>(st.grp) * p.splits + split;
    if (st.grp_ok && row_in_tile % R == 0 && CPMTP_INDEX_OK(ti, 1, static_cast<size_t>(p.groups) * p.splits)) {
      p.part_tm[ti] = m;
      p.part_tl[ti] = l;
    }
  }
  __device__ static void tile(const Params& p, State& st, uint32_t tacc, int, int n_tile, int row_in_tile,
                              uint8_t*, int) {
    const int sub = row_in_tile % R;
    const uint16_t* trow = p.T + static_cast<size_t>(st.grp_ok ? st.grp : 0) * p.V;
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
      const int col0 = n_tile * BN + c;
      if (col0 >= p.V) break;   // uniform across the CTA
      float e[32], w[32];
      ptx::tmem_ld_32x32(tacc + c, e);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j) e[j] = ptx::ex2_approx(fmaf(e[j], kLog2e, st.c2));
      if (col0 + 32 > p.V) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (col0 + j >= p.V) e[j] = 0.f;
      }
#pragma unroll
      for (int j = 0; j < 32; ++j) w[j] = e[j];
      GL::reduce_scatter(w, sub);
      finish_columns<GL::W, true>(w, trow, col0 + sub * GL::W, p.V, st.grp_ok, p.vec != 0, 0.f, &st.tm2, &st.tl);
      GL::all_gather(w, sub);
      float sum = 0.f;
#pragma unroll
      for (int j = 0; j < 32; ++j) sum = fmaf(e[j], w[j], sum);
      st.acc += sum;
    }
  }
};

// ---------------------------------------------------------------------------
// Backward: logit gradient of  sum up * prefix + sum uk * kl  for a chunk of groups,
//   G[(g,a), v] = coef (1[v = x_g] - P(v)) + uk_g (e(v) l(v) - P(v) pm[(g,a)]),
// bf16, written at ORIGINAL rows relative to the chunk.  Columns in [V, ldg) are zero.
struct DistillGradParams {
  uint16_t* G;            // [groups * r, ldg] bf16 (this chunk)
  const float* lse;       // the arrays below are indexed by GLOBAL row / group
  const float* coef;      // [.., r]  d objective / d C  (cross-entropy and KL-weight paths)
  const float* logpi;
  const float* pm;
  const float* uk;        // [groups_total]
  const float* lse_t;     // [groups_total]
  const uint16_t* T;      // [groups_total, V]
  const int32_t* x;       // [groups_total]
  long long grp0;         // first group of the chunk
  int groups, r, V, ldg, vec;
};

template <int BN, int R>
struct EpiDistillGrad : EpiDefaults {
  using Params = DistillGradParams;
  struct State { float lse2, pi, coef, ukpi, ckm, lt; long long grp, orow_local; int tok; bool valid, grp_ok; };
  using GL = GroupLanes<R>;
  __device__ static void unit_begin(const Params& p, State& st, int m_tile, int, int row_in_tile) {
    const int gl = m_tile * (kBM / R) + row_in_tile / R;
    const int a = row_in_tile % R;
    st.grp_ok = gl < p.groups;
    st.valid = st.grp_ok && a < p.r;
    st.grp = p.grp0 + gl;
    st.orow_local = static_cast<long long>(gl) * p.r + a;
    st.lse2 = INFINITY;   // P = 0 for padding rows
    st.pi = st.coef = st.ukpi = st.ckm = st.lt = 0.f;
    st.tok = -1;
    if (st.grp_ok) st.lt = p.lse_t[st.grp];
    if (st.valid) {
      const long long orow = st.grp * p.r + a;
      const float uk = p.uk[st.grp];
      st.lse2 = p.lse[orow] * kLog2e;
      st.pi = __expf(p.logpi[orow]);
      st.coef = p.coef[orow];
      st.ukpi = uk * st.pi;
      st.ckm = st.coef + uk * p.pm[orow];
      const int tok = p.x[st.grp];
      st.tok = tok < 0 ? 0 : (tok >= p.V ? p.V - 1 : tok);
    }
  }
  __device__ static void unit_end(const Params&, State&, int, int, int, uint8_t*, int) {}
  __device__ static void tile(const Params& p, State& st, uint32_t tacc, int, int n_tile, int row_in_tile,
                              uint8_t*, int) {
    const int sub = row_in_tile % R;
    const uint16_t* trow = p.T + static_cast<size_t>(st.grp_ok ? st.grp : 0) * p.V;
#pragma unroll 1
    for (int c = 0; c < BN; c += 32) {
      const int col0 = n_tile * BN + c;
      if (col0 >= p.ldg) break;   // uniform across the CTA
      float v[32], w[32];
      ptx::tmem_ld_32x32(tacc + c, v);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = ptx::ex2_approx(fmaf(v[j], kLog2e, -st.lse2));
      if (col0 + 32 > p.V) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (col0 + j >= p.V) v[j] = 0.f;
      }
#pragma unroll
      for (int j = 0; j < 32; ++j) w[j] = st.pi * v[j];
      GL::reduce_scatter(w, sub);
      finish_columns<GL::W>(w, trow, col0 + sub * GL::W, p.V, st.grp_ok, p.vec != 0, st.lt);
      GL::all_gather(w, sub);
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] *= fmaf(st.ukpi, w[j], -st.ckm);
      const int t = st.tok - col0;
      if (t >= 0 && t < 32) {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (j == t) v[j] += st.coef;
      }
      const size_t gi = static_cast<size_t>(st.orow_local) * p.ldg + col0;
      if (st.valid && CPMTP_INDEX_OK(gi, 32, static_cast<size_t>(p.groups) * p.r * p.ldg)) store_bf16x32(p.G + gi, v);
    }
  }
};

}  // namespace cpmtp
