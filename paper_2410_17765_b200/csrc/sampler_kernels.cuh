// Draft generation from the factors (sampling section of the paper).
//
// The unembedding GEMM has stored the logits S[(i,k), v] (fp32) and their
// logsumexp; token s of the draft is then chosen from
//   mix[v] = log sum_alpha b_alpha * P^(s)(v | alpha),
//   b_alpha = w_alpha * prod_{t<s} P^(t)(x_t | alpha)          (Eq. 11 for s = 1),
// either greedily or by the Gumbel-max rule on caller-supplied uniforms, and the
// k most likely tokens are reported as candidates for a static draft tree.
// One streaming kernel per token: every block scans a chunk of the vocabulary for one position
// and leaves its k best tokens; the block that finishes a position last (a counter in global
// memory, no waiting anywhere) merges the chunks and folds the chosen token's factors into b.
// The reported log-probabilities (joint and candidates'), which no later selection needs, are
// recomputed from the unrounded z by a few blocks of the next launch.  Ties go to the lowest
// token id, so results are reproducible.
#pragma once
#include <cstdint>

#include "../../include/cpmtp.h"
#include "small_kernels.cuh"
#include "tc_gemm.cuh"

namespace cpmtp {

constexpr int kMaxTopk = 8;
constexpr int kSampleThreads = 256;
constexpr int kSampleWarps = kSampleThreads / 32;
constexpr int kSamplePerThread = 8;                                // vocabulary entries per thread: two groups of four
constexpr int kSampleChunk = kSampleThreads * kSamplePerThread;   // vocabulary entries per block
constexpr int kSampleBlocksPerSm = 4;                              // 64 registers per thread: a whole step is one wave
static_assert(kSamplePerThread == kMaxTopk, "a thread's entries are its candidate list");

struct __align__(8) Cand {
  float score;
  int idx;
};
constexpr int kNoToken = 0x7fffffff;

// Read a candidate that another block wrote during this launch (L2, not this SM's L1).
__device__ __forceinline__ Cand load_cand_cg(const Cand* p) {
  const int2 raw = __ldcg(reinterpret_cast<const int2*>(p));
  return Cand{__int_as_float(raw.x), raw.y};
}

__device__ __forceinline__ bool cand_better(float s1, int i1, float s2, int i2) {
  return s1 > s2 || (s1 == s2 && i1 < i2);
}

// List of at most kMaxTopk candidates kept in registers.  insert() expects the list in order (best first) and
// keeps it so; the other members accept any order.
struct TopList {
  float score[kMaxTopk];
  int idx[kMaxTopk];
  __device__ void init() {
#pragma unroll
    for (int j = 0; j < kMaxTopk; ++j) {
      score[j] = -INFINITY;
      idx[j] = kNoToken;
    }
  }
  // The lane's best entry (entries need not be in order; among equal scores the lowest id).
  __device__ Cand best() const {
    Cand b{score[0], idx[0]};
#pragma unroll
    for (int j = 1; j < kMaxTopk; ++j)
      if (cand_better(score[j], idx[j], b.score, b.idx)) b = Cand{score[j], idx[j]};
    return b;
  }
  // Empty the entry that holds token id `i` (ids are unique).
  __device__ void remove(int i) {
#pragma unroll
    for (int j = 0; j < kMaxTopk; ++j)
      if (idx[j] == i) {
        score[j] = -INFINITY;
        idx[j] = kNoToken;
      }
  }
  __device__ void insert(float s, int i, int k) {
    float last_s = -INFINITY;
    int last_i = kNoToken;
#pragma unroll
    for (int j = 0; j < kMaxTopk; ++j)   // constant indices only: the lists stay in registers
      if (j == k - 1) {
        last_s = score[j];
        last_i = idx[j];
      }
    if (!cand_better(s, i, last_s, last_i)) return;
#pragma unroll
    for (int j = kMaxTopk - 1; j >= 0; --j) {
      if (j >= k) continue;
      const bool here = cand_better(s, i, score[j], idx[j]);
      const bool above = j > 0 && cand_better(s, i, score[j - 1], idx[j - 1]);
      if (here && above) {           // shift down
        score[j] = score[j - 1];
        idx[j] = idx[j - 1];
      } else if (here) {
        score[j] = s;
        idx[j] = i;
      }
    }
  }
};

// Warp-wide best candidate (score desc, index asc), the same in every lane: two hardware warp reductions on
// integers, the maximum of the scores mapped to unsigned keys of the same order, then the lowest id among
// the lanes that hold it.  Scores are never NaN.
__device__ __forceinline__ unsigned int order_key(float x) {
  const unsigned int b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_value(unsigned int k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
__device__ __forceinline__ Cand warp_best(Cand c) {
  const unsigned int key = order_key(c.score);
  const unsigned int top = __reduce_max_sync(0xffffffffu, key);
  const int idx = __reduce_min_sync(0xffffffffu, key == top ? c.idx : kNoToken);
  return Cand{key_value(top), idx};
}

// Block-wide best candidate (score desc, index asc); result valid in every thread.
__device__ __forceinline__ Cand block_best(Cand c, Cand* red /* [kSampleWarps] shared */) {
  c = warp_best(c);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();
  if (lane == 0) red[warp] = c;
  __syncthreads();
  return warp_best(lane < kSampleWarps ? red[lane] : Cand{-INFINITY, kNoToken});
}

// The k best entries over the lists of a warp's lanes, which it empties as it goes (token ids are unique, so
// every round has one winner): lane t < k returns the t-th best, the other lanes an empty candidate.
__device__ __forceinline__ Cand warp_topk(TopList& mine, int k) {
  const int lane = threadIdx.x & 31;
  Cand res{-INFINITY, kNoToken};
  Cand c = mine.best();
  for (int round = 0; round < k; ++round) {
    const Cand w = warp_best(c);
    if (w.idx == c.idx && c.idx != kNoToken) {   // this lane held the winner: its next best comes up
      mine.remove(w.idx);
      c = mine.best();
    }
    if (lane == round) res = w;
  }
  return res;
}

// The k best entries over the lists of all threads of the block (emptied on the way), written best first to
// out[0..k) (shared or global) by warp 0: every warp reduces its lanes' lists to one list, then warp 0 does
// the same with the warps' lists (lane w holds warp w's).  `stage` is shared scratch of kSampleWarps * kMaxTopk candidates.
// Ends with a barrier.  Exhaustive: block_topk below falls back on it when many entries tie.
__device__ __forceinline__ void block_topk_merge(TopList& mine, int k, Cand* out, Cand* stage) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const Cand w = warp_topk(mine, k);
  __syncthreads();   // `stage` may still be read from a previous use
  if (lane < k) stage[warp * kMaxTopk + lane] = w;
  __syncthreads();
  if (warp == 0) {
    TopList merged;
    merged.init();
    if (lane < kSampleWarps) {
#pragma unroll
      for (int j = 0; j < kMaxTopk; ++j)
        if (j < k) {
          const Cand c = stage[lane * kMaxTopk + j];
          merged.score[j] = c.score;
          merged.idx[j] = c.idx;
        }
    }
    const Cand f = warp_topk(merged, k);
    if (lane < k) out[lane] = f;
  }
  __syncthreads();
}

// Shared scratch of block_topk.
constexpr int kSelectCap = 64;
static_assert(kSampleWarps * kMaxTopk == 64, "block_topk reads the warps' maxima as two per lane");
struct SelectScratch {
  unsigned int wkeys[kSampleWarps * kMaxTopk];   // every warp's k largest lane maxima (as order keys)
  unsigned int bound;                            // the k-th largest lane maximum of the block
  int count;
  Cand cand[kSelectCap];
  Cand stage[kSampleWarps * kMaxTopk];           // block_topk_merge
};

// The k best entries over the lists of all threads of the block, written best first to out[0..k) (shared or
// global) by warp 0; ends with a barrier.  Instead of merging lists, a bound is found first: the k-th largest of
// the threads' own maxima.  k different threads hold an entry at least that good, so the k-th best entry of the
// block is no worse, and every entry not below the bound (usually just the k winners) goes into a small
// candidate array from which one warp picks the k best by (score desc, id asc).  The order in which candidates
// arrive does not matter, so the result is reproducible.  More than kSelectCap entries at or above the bound
// (long runs of equal scores): the exhaustive merge.  Keys of real entries are > 0; 0 stands for "none".
__device__ __forceinline__ void block_topk(TopList& mine, int k, Cand* out, SelectScratch* sc) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned int key[kMaxTopk];
  unsigned int cur = 0u;
#pragma unroll
  for (int j = 0; j < kMaxTopk; ++j) {
    key[j] = mine.idx[j] != kNoToken ? order_key(mine.score[j]) : 0u;
    cur = max(cur, key[j]);
  }
  for (int round = 0; round < k; ++round) {   // the warp's k largest thread maxima, one per round
    const unsigned int top = __reduce_max_sync(0xffffffffu, cur);
    const unsigned int holders = __ballot_sync(0xffffffffu, cur == top);
    if (lane == __ffs(holders) - 1) cur = 0u;
    if (lane == 0) sc->wkeys[warp * kMaxTopk + round] = top;
  }
  if (threadIdx.x == 0) sc->count = 0;
  __syncthreads();
  if (warp == 0) {   // the k-th largest of all warps' lists: lane holds entries lane and lane + 32 of [warps][kMaxTopk]
    unsigned int a0 = (lane & (kMaxTopk - 1)) < k ? sc->wkeys[lane] : 0u;
    unsigned int a1 = (lane & (kMaxTopk - 1)) < k ? sc->wkeys[lane + 32] : 0u;
    unsigned int top = 0u;
    for (int round = 0; round < k; ++round) {
      const unsigned int m = max(a0, a1);
      top = __reduce_max_sync(0xffffffffu, m);
      const unsigned int holders = __ballot_sync(0xffffffffu, m == top);
      if (lane == __ffs(holders) - 1) {
        if (a0 == top) a0 = 0u; else a1 = 0u;
      }
    }
    if (lane == 0) sc->bound = top;
  }
  __syncthreads();
  const unsigned int bound = sc->bound;
#pragma unroll
  for (int j = 0; j < kMaxTopk; ++j)
    if (key[j] != 0u && key[j] >= bound) {
      const int pos = atomicAdd(&sc->count, 1);
      if (pos < kSelectCap) sc->cand[pos] = Cand{mine.score[j], mine.idx[j]};
    }
  __syncthreads();
  const int cnt = sc->count;
  if (cnt > kSelectCap) {
    block_topk_merge(mine, k, out, sc->stage);
    return;
  }
  if (warp == 0) {
    Cand c0 = lane < cnt ? sc->cand[lane] : Cand{-INFINITY, kNoToken};
    Cand c1 = lane + 32 < cnt ? sc->cand[lane + 32] : Cand{-INFINITY, kNoToken};
    Cand res{-INFINITY, kNoToken};
    for (int round = 0; round < k; ++round) {
      const bool first = cand_better(c0.score, c0.idx, c1.score, c1.idx);
      const Cand m = first ? c0 : c1;
      const Cand w = warp_best(m);
      if (w.idx == m.idx && m.idx != kNoToken) {
        if (first) c0 = Cand{-INFINITY, kNoToken}; else c1 = Cand{-INFINITY, kNoToken};
      }
      if (lane == round) res = w;
    }
    if (lane < k) out[lane] = res;
  }
  __syncthreads();
}

// mix[j] = logsumexp_a(S[a, v + j] + off[a]) for the four vocabulary entries v .. v + 3 (16-byte aligned row
// pieces); off2 = off * log2(e), and the sums run in the log2 domain.  Up to eight experts (`fetched`): the rows
// were fetched into q by fetch_four and both passes (maximum, sum of exponentials) run from registers; more
// experts: two passes over memory, the second of which hits the caches.
__device__ __forceinline__ void fetch_four(const float* __restrict__ Srow, int lds, int v, int r, float4 (&q)[8]) {
#pragma unroll
  for (int a = 0; a < 8; ++a)
    if (a < r) q[a] = __ldg(reinterpret_cast<const float4*>(Srow + static_cast<size_t>(a) * lds + v));
}
__device__ __forceinline__ void mix_of_four(const float* __restrict__ Srow, int lds, int v, int r, bool fetched,
                                            float4 (&q)[8], const float* off2_s, float (&mix)[4]) {
  constexpr float kL2e = 1.4426950408889634f, kLn2f = 0.6931471805599453f;
  float m[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
  float l[4] = {0.f, 0.f, 0.f, 0.f};
  if (fetched) {
#pragma unroll
    for (int a = 0; a < 8; ++a)
      if (a < r) {
        const float off = off2_s[a];
        q[a].x = fmaf(q[a].x, kL2e, off); q[a].y = fmaf(q[a].y, kL2e, off);
        q[a].z = fmaf(q[a].z, kL2e, off); q[a].w = fmaf(q[a].w, kL2e, off);
        m[0] = fmaxf(m[0], q[a].x); m[1] = fmaxf(m[1], q[a].y);
        m[2] = fmaxf(m[2], q[a].z); m[3] = fmaxf(m[3], q[a].w);
      }
#pragma unroll
    for (int a = 0; a < 8; ++a)
      if (a < r) {
        l[0] += ptx::ex2_approx(q[a].x - m[0]); l[1] += ptx::ex2_approx(q[a].y - m[1]);
        l[2] += ptx::ex2_approx(q[a].z - m[2]); l[3] += ptx::ex2_approx(q[a].w - m[3]);
      }
  } else {
#pragma unroll 4
    for (int a = 0; a < r; ++a) {
      const float4 w = __ldg(reinterpret_cast<const float4*>(Srow + static_cast<size_t>(a) * lds + v));
      const float off = off2_s[a];
      m[0] = fmaxf(m[0], fmaf(w.x, kL2e, off)); m[1] = fmaxf(m[1], fmaf(w.y, kL2e, off));
      m[2] = fmaxf(m[2], fmaf(w.z, kL2e, off)); m[3] = fmaxf(m[3], fmaf(w.w, kL2e, off));
    }
#pragma unroll 4
    for (int a = 0; a < r; ++a) {
      const float4 w = __ldg(reinterpret_cast<const float4*>(Srow + static_cast<size_t>(a) * lds + v));
      const float off = off2_s[a];
      l[0] += ptx::ex2_approx(fmaf(w.x, kL2e, off) - m[0]); l[1] += ptx::ex2_approx(fmaf(w.y, kL2e, off) - m[1]);
      l[2] += ptx::ex2_approx(fmaf(w.z, kL2e, off) - m[2]); l[3] += ptx::ex2_approx(fmaf(w.w, kL2e, off) - m[3]);
    }
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) mix[j] = (m[j] + ptx::lg2_approx(l[j])) * kLn2f;
}

// Exact logits of one token for all r experts of draft step s at position i, from the unrounded z:
//   out[a] = E[tok, :] . z32[(i, s, a), :] - lse[(i, s, a)],   a < r,
// computed by the whole block (four experts at a time; every thread takes 8-element pieces of the rows).
// `red` is shared scratch of kSampleWarps * CPMTP_MAX_R floats.  d % 64 == 0; rows are 16-byte aligned.
// Ends with a barrier, after which out[0..r) is valid in shared memory.
__device__ __forceinline__ void block_token_logits(const uint16_t* __restrict__ E, int tok, const float* __restrict__ z32,
                                                   const float* __restrict__ lse, size_t row0, int d, int r,
                                                   float* out, float* red) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint4* erow = reinterpret_cast<const uint4*>(E + static_cast<size_t>(tok) * d);
  for (int a0 = 0; a0 < r; a0 += 4) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int g = threadIdx.x; g < (d >> 3); g += kSampleThreads) {
      // all nine loads of this piece are issued before the first is used (experts beyond r re-read expert
      // r - 1 and are dropped below), so the piece costs one round trip to memory, not five
      const uint4 e = __ldg(erow + g);
      float4 z0[4], z1[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int a = min(a0 + u, r - 1);
        const float4* zrow = reinterpret_cast<const float4*>(z32 + (row0 + a) * d);
        z0[u] = __ldg(zrow + 2 * g);
        z1[u] = __ldg(zrow + 2 * g + 1);
      }
      const float e0 = ptx::bf16_lo(e.x), e1 = ptx::bf16_hi(e.x), e2 = ptx::bf16_lo(e.y), e3 = ptx::bf16_hi(e.y);
      const float e4 = ptx::bf16_lo(e.z), e5 = ptx::bf16_hi(e.z), e6 = ptx::bf16_lo(e.w), e7 = ptx::bf16_hi(e.w);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        float t = acc[u];
        t = fmaf(e0, z0[u].x, t); t = fmaf(e1, z0[u].y, t); t = fmaf(e2, z0[u].z, t); t = fmaf(e3, z0[u].w, t);
        t = fmaf(e4, z1[u].x, t); t = fmaf(e5, z1[u].y, t); t = fmaf(e6, z1[u].z, t); t = fmaf(e7, z1[u].w, t);
        acc[u] = t;
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const float t = warp_sum(acc[u]);
      if (lane == 0 && a0 + u < r) red[warp * CPMTP_MAX_R + a0 + u] = t;
    }
  }
  __syncthreads();
  if (threadIdx.x < r) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < kSampleWarps; ++w) t += red[w * CPMTP_MAX_R + threadIdx.x];
    out[threadIdx.x] = t - lse[row0 + threadIdx.x];
  }
  __syncthreads();
}

// The reported values of draft step s at position i, from the unrounded z, which no later selection depends on.
// Job j < topk:  topk_logp[i, s, j] = logsumexp_a(log b_a + log P^(s)(cand_j | a)) - logsumexp_a log b_a, with b the
// exact expert weights before step s (lb_exact[s]).  Job j == topk: fold the chosen token into the exact weights,
// lb_exact[s + 1] = lb_exact[s] + log P^(s)(token | .), and after the last step write the joint log-probability.
// This block takes jobs first, first + stride, ...; tok_hist holds kMaxTopk candidates and then the chosen token.
__device__ __forceinline__ void exact_step_values(const uint16_t* __restrict__ E, const float* __restrict__ z32,
                                                  const float* __restrict__ lse, float* __restrict__ lb_exact,
                                                  const int* __restrict__ tok_hist, int i, int s, int d, int N, int V, int n,
                                                  int r, int topk, int first, int stride, float* __restrict__ topk_logp,
                                                  float* __restrict__ logp_joint, float* tgt_s, float* red) {
  const size_t row0 = (static_cast<size_t>(i) * n + s) * r;
  const float* lb_before = lb_exact + (static_cast<size_t>(s) * N + i) * r;
  float* lb_after = lb_exact + (static_cast<size_t>(s + 1) * N + i) * r;
  const int* toks = tok_hist + (static_cast<size_t>(s) * N + i) * (kMaxTopk + 1);
  for (int j = first; j <= topk; j += stride) {
    const bool chosen = j == topk;
    if (!chosen && topk_logp == nullptr) continue;
    // a token outside the vocabulary would gather from beyond E (checked build: reported, row 0 read instead)
    int tok = toks[chosen ? kMaxTopk : j];
    if (!CPMTP_INDEX_OK(tok, 1, V)) tok = 0;
    block_token_logits(E, tok, z32, lse, row0, d, r, tgt_s, red);
    if (threadIdx.x < 32) {
      const int a = threadIdx.x;
      const float b = a < r ? lb_before[a] : -INFINITY;
      const float x = a < r ? b + tgt_s[a] : -INFINITY;
      const float m = warp_max(x);
      const float lp = m + logf(warp_sum(a < r ? expf(x - m) : 0.f));
      if (chosen) {
        if (a < r) lb_after[a] = x;
        if (s == n - 1 && logp_joint != nullptr && a == 0) logp_joint[i] = lp;
      } else {
        const float mb = warp_max(b);
        const float norm = mb + logf(warp_sum(a < r ? expf(b - mb) : 0.f));
        if (a == 0) topk_logp[(static_cast<size_t>(i) * n + s) * topk + j] = lp - norm;
      }
    }
    __syncthreads();   // tgt_s and red are reused by the next job
  }
}

// One draft step.  Grid (chunks, N), kSampleThreads threads.
//   lb_sel   [n + 1][N][r]  expert weights as the SELECTION sees them before every step: the chosen tokens' factors
//                           are read from the stored logits S (computed from bf16-rounded z, like all of S)
//   lb_exact [n + 1][N][r]  the same from the unrounded z: what the reported log-probabilities are made of
//   tok_hist [n][N][kMaxTopk + 1]  candidate tokens of every step, then the chosen one
//   phase 1 (every block): scan the chunk's entries of position i, mix[v] = logsumexp_a(log b_a + S[s,a,v] - lse[s,a]);
//            keep the k best tokens and, when sampling, the best Gumbel-perturbed score; write them to part_*.
//   phase 2 (the block that raises done[i] to the chunk count, i.e. the last to finish for position i): merge the
//            chunks, choose the token, fold its stored logits into lb_sel for the next step, and reset done[i].
//   side jobs (blocks with chunk <= topk, after their own part): the exact values of the PREVIOUS step (see
//            exact_step_values), which nothing on the selection path waits for; draft_tail_kernel does the same for
//            the last step.
// No block waits for another: whichever finishes last does the merge.
__global__ void __launch_bounds__(kSampleThreads, kSampleBlocksPerSm)
draft_step_kernel(const float* __restrict__ S, int lds, const float* __restrict__ z32, const uint16_t* __restrict__ E,
                  int d, const float* __restrict__ lse, float* __restrict__ lb_sel, float* __restrict__ lb_exact,
                  const float* __restrict__ uniform, float inv_temp, int s, int N, int V, int n, int r, int topk,
                  const int32_t* __restrict__ forced, Cand* __restrict__ part_top, Cand* __restrict__ part_best,
                  unsigned int* __restrict__ done, int* __restrict__ tok_hist, int* __restrict__ dev_status,
                  int32_t* __restrict__ draft, float* __restrict__ logp_joint, int32_t* __restrict__ topk_tokens,
                  float* __restrict__ topk_logp) {
  __shared__ float off_s[CPMTP_MAX_R];
  __shared__ float lb_s[CPMTP_MAX_R];
  __shared__ float tgt_s[CPMTP_MAX_R];                  // log P^(s)(token | expert)
  __shared__ float red_f[kSampleWarps * CPMTP_MAX_R];
  __shared__ float norm_s;
  __shared__ Cand red[kSampleWarps];
  __shared__ SelectScratch select;
  __shared__ Cand final_top[kMaxTopk];
  __shared__ int tok_s;
  __shared__ bool is_last;
  const int chunk = blockIdx.x, chunks = gridDim.x, i = blockIdx.y;
  const int K = n * r;
  // Launched with programmatic stream serialization: the next step's blocks may become resident while this
  // step's last blocks still merge.  What they do before grid_dep_wait() touches only the stored logits, which
  // no draft step writes: the first half of the scan's loads is in flight while the step before finishes.
  ptx::grid_dep_launch();
  const float* Srow = S + (static_cast<size_t>(i) * K + static_cast<size_t>(s) * r) * lds;
  const int v_end = min(V, (chunk + 1) * kSampleChunk);
  const bool fetched = r <= 8;
  float4 q[8];
  {
    const int v0 = chunk * kSampleChunk + 4 * threadIdx.x;
    if (fetched && v0 < v_end) fetch_four(Srow, lds, v0, r, q);
  }
  ptx::grid_dep_wait();
  const float* lb = lb_sel + static_cast<size_t>(s) * N * r;              // before this step
  float* lb_next = lb_sel + static_cast<size_t>(s + 1) * N * r;           // after it
  if (threadIdx.x < 32) {
    const int a = threadIdx.x;
    const float b = a < r ? lb[static_cast<size_t>(i) * r + a] : -INFINITY;
    if (a < r) {
      lb_s[a] = b;
      off_s[a] = (b - lse[static_cast<size_t>(i) * K + s * r + a]) * 1.4426950408889634f;   // log2 domain
    }
    const float m = warp_max(b);
    const float e = a < r ? expf(b - m) : 0.f;
    const float tot = warp_sum(e);
    if (a == 0) norm_s = m + logf(tot);   // log sum_alpha b_alpha before this token is folded in
  }
  __syncthreads();
  const float norm = norm_s;
  // ---- phase 1: this block's chunk
  {
    const float* urow = uniform != nullptr ? uniform + (static_cast<size_t>(i) * n + s) * V : nullptr;
    TopList top;
    top.init();
    Cand best{-INFINITY, kNoToken};
    // two groups of four consecutive vocabulary entries per thread, half a chunk apart (lds % 32 == 0: 16-byte
    // aligned loads, a warp reads 512 contiguous bytes of every row; entries in [V, lds) exist in the buffer
    // and are left out below)
#pragma unroll
    for (int grp = 0; grp < 2; ++grp) {
      const int v0 = chunk * kSampleChunk + grp * (kSampleChunk / 2) + 4 * threadIdx.x;
      if (v0 >= v_end) continue;
      float mix[4];
      if (grp == 1 && fetched) fetch_four(Srow, lds, v0, r, q);   // (the first group's rows were fetched above)
      mix_of_four(Srow, lds, v0, r, fetched, q, off_s, mix);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int v = v0 + j;
        if (v >= v_end) continue;
        top.score[grp * 4 + j] = mix[j];
        top.idx[grp * 4 + j] = v;
        float sc = mix[j];
        if (urow != nullptr) sc = (mix[j] - norm) * inv_temp - logf(-logf(urow[v]));
        if (cand_better(sc, v, best.score, best.idx)) best = Cand{sc, v};
      }
    }
    block_topk(top, topk, part_top + (static_cast<size_t>(i) * chunks + chunk) * kMaxTopk, &select);
    if (urow != nullptr) {
      const Cand b = block_best(best, red);
      if (threadIdx.x == 0) part_best[static_cast<size_t>(i) * chunks + chunk] = b;
    }
  }
  // ---- who is last for this position?
  __threadfence();   // this block's partial results are visible device-wide before the counter moves
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int prev = atomicAdd(done + i, 1u);
    is_last = prev + 1u == static_cast<unsigned int>(chunks);
  }
  __syncthreads();
  if (is_last) {
    __threadfence();   // the other blocks' partial results, published before their increments, are read below
    // ---- phase 2: merge (thread t holds the lists of chunks t, t + 256, ..., each written best first), choose, fold
    TopList top;
    top.init();
    Cand best{-INFINITY, kNoToken};
    for (int c = threadIdx.x; c < chunks; c += kSampleThreads) {
      const Cand* src = part_top + (static_cast<size_t>(i) * chunks + c) * kMaxTopk;
      Cand got[kMaxTopk];
#pragma unroll
      for (int j = 0; j < kMaxTopk; ++j) got[j] = j < topk ? load_cand_cg(src + j) : Cand{-INFINITY, kNoToken};
      if (c == static_cast<int>(threadIdx.x)) {   // the thread's first list is taken as it is
#pragma unroll
        for (int j = 0; j < kMaxTopk; ++j) {
          top.score[j] = got[j].score;
          top.idx[j] = got[j].idx;
        }
      } else {
#pragma unroll
        for (int j = 0; j < kMaxTopk; ++j)
          if (got[j].idx != kNoToken) top.insert(got[j].score, got[j].idx, topk);
      }
      if (uniform != nullptr) {
        const Cand pb = load_cand_cg(part_best + static_cast<size_t>(i) * chunks + c);
        if (cand_better(pb.score, pb.idx, best.score, best.idx)) best = pb;
      }
    }
    block_topk(top, topk, final_top, &select);
    if (uniform != nullptr) best = block_best(best, red);
    if (threadIdx.x == 0) {   // the drafted token: the caller's, if one is given for this step
      int tok = uniform != nullptr ? best.idx : final_top[0].idx;
      if (forced != nullptr) {
        const int f = forced[static_cast<size_t>(i) * n + s];
        if (f >= V) {
          if (dev_status != nullptr) atomicMax(dev_status, 1);   // out of range: clamped and reported
          tok = V - 1;
        } else if (f >= 0) {
          tok = f;
        }
      }
      if (!CPMTP_INDEX_OK(tok, 1, V)) tok = 0;
      tok_s = tok;
      draft[static_cast<size_t>(i) * n + s] = tok;
      tok_hist[(static_cast<size_t>(s) * N + i) * (kMaxTopk + 1) + kMaxTopk] = tok;
      done[i] = 0u;   // ready for the next step (launches on the stream are ordered)
    }
    if (threadIdx.x < topk) {
      const int t = final_top[threadIdx.x].idx;
      tok_hist[(static_cast<size_t>(s) * N + i) * (kMaxTopk + 1) + threadIdx.x] = t;
      if (topk_tokens != nullptr) topk_tokens[(static_cast<size_t>(i) * n + s) * topk + threadIdx.x] = t;
    }
    __syncthreads();
    if (threadIdx.x < r)   // the chosen token's factors as the selection sees them: its stored logits
      lb_next[static_cast<size_t>(i) * r + threadIdx.x] =
          lb_s[threadIdx.x] + __ldg(Srow + static_cast<size_t>(threadIdx.x) * lds + tok_s) -
          lse[static_cast<size_t>(i) * K + s * r + threadIdx.x];
  }
  // ---- side jobs: the exact values of the previous step
  if (s > 0 && chunk <= topk && (topk_logp != nullptr || logp_joint != nullptr)) {
    __syncthreads();
    exact_step_values(E, z32, lse, lb_exact, tok_hist, i, s - 1, d, N, V, n, r, topk, chunk, chunks, topk_logp, logp_joint,
                      tgt_s, red_f);
  }
#ifdef CPMTP_DEBUG
  if (threadIdx.x == 0 && dev_status != nullptr) {
    const int seen = *const_cast<volatile int*>(&g_debug_status);
    if (seen != 0) atomicMax(dev_status, seen);
  }
#endif
}

// The exact values of the last draft step.  Grid (min(topk + 1, anything >= 1), N).
__global__ void __launch_bounds__(kSampleThreads, kSampleBlocksPerSm)
draft_tail_kernel(const float* __restrict__ z32, const uint16_t* __restrict__ E, int d, const float* __restrict__ lse,
                  float* __restrict__ lb_exact, const int* __restrict__ tok_hist, int N, int V, int n, int r, int topk,
                  float* __restrict__ topk_logp, float* __restrict__ logp_joint) {
  __shared__ float tgt_s[CPMTP_MAX_R];
  __shared__ float red_f[kSampleWarps * CPMTP_MAX_R];
  ptx::grid_dep_wait();   // the last step's tokens come from the launch before this one
  exact_step_values(E, z32, lse, lb_exact, tok_hist, blockIdx.y, n - 1, d, N, V, n, r, topk, blockIdx.x, gridDim.x,
                    topk_logp, logp_joint, tgt_s, red_f);
}

// Draft verification: one thread per position.
__global__ void verify_draft_kernel(const int32_t* __restrict__ draft, const int32_t* __restrict__ base_tokens,
                                    const float* __restrict__ logp_prefix, const float* __restrict__ logp_base,
                                    const float* __restrict__ uniform, int32_t* __restrict__ accepted, int N, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  int k = 0;
  if (base_tokens != nullptr) {
    while (k < n && draft[static_cast<size_t>(i) * n + k] == base_tokens[static_cast<size_t>(i) * n + k]) ++k;
  } else {
    float prev = 0.f;
    while (k < n) {
      const float pre = logp_prefix[static_cast<size_t>(i) * n + k];
      const float ratio = expf(logp_base[static_cast<size_t>(i) * n + k] - (pre - prev));
      if (!(uniform[static_cast<size_t>(i) * n + k] < fminf(1.f, ratio))) break;
      prev = pre;
      ++k;
    }
  }
  accepted[i] = k;
}

}  // namespace cpmtp
