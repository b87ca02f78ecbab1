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
// The candidates' reported log-probabilities, which no later step needs, are computed by a few
// blocks of the next launch.  Ties go to the lowest token id, so results are reproducible.
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
static_assert(kSamplePerThread == kMaxTopk, "a thread's sorted entries are its candidate list");

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

// Sorted (best first) list of at most kMaxTopk candidates kept in registers.
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
  // Put all eight entries in order with a 19-comparator sorting network (constant indices only).
  __device__ void sort() {
#define CPMTP_CSWAP(a, b)                                          \
  if (cand_better(score[b], idx[b], score[a], idx[a])) {           \
    const float ts = score[a]; score[a] = score[b]; score[b] = ts; \
    const int ti = idx[a]; idx[a] = idx[b]; idx[b] = ti;           \
  }
    CPMTP_CSWAP(0, 1) CPMTP_CSWAP(2, 3) CPMTP_CSWAP(4, 5) CPMTP_CSWAP(6, 7)
    CPMTP_CSWAP(0, 2) CPMTP_CSWAP(1, 3) CPMTP_CSWAP(4, 6) CPMTP_CSWAP(5, 7)
    CPMTP_CSWAP(1, 2) CPMTP_CSWAP(5, 6)
    CPMTP_CSWAP(0, 4) CPMTP_CSWAP(1, 5) CPMTP_CSWAP(2, 6) CPMTP_CSWAP(3, 7)
    CPMTP_CSWAP(2, 4) CPMTP_CSWAP(3, 5)
    CPMTP_CSWAP(1, 2) CPMTP_CSWAP(3, 4) CPMTP_CSWAP(5, 6)
#undef CPMTP_CSWAP
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

__device__ __forceinline__ Cand warp_best(Cand c) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float os = __shfl_xor_sync(0xffffffffu, c.score, o);
    const int oi = __shfl_xor_sync(0xffffffffu, c.idx, o);
    if (cand_better(os, oi, c.score, c.idx)) {
      c.score = os;
      c.idx = oi;
    }
  }
  return c;
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

// The k best entries over the sorted lists of a warp's lanes (token ids are unique, so every round
// has one winner): lane t < k returns the t-th best, the other lanes an empty candidate.
__device__ __forceinline__ Cand warp_topk(const TopList& mine, int k) {
  const int lane = threadIdx.x & 31;
  int head = 0;
  Cand res{-INFINITY, kNoToken};
  for (int round = 0; round < k; ++round) {
    Cand c{-INFINITY, kNoToken};
#pragma unroll
    for (int j = 0; j < kMaxTopk; ++j)
      if (j == head) c = Cand{mine.score[j], mine.idx[j]};
    const Cand w = warp_best(c);
    if (w.idx == c.idx && c.idx != kNoToken) ++head;
    if (lane == round) res = w;
  }
  return res;
}

// The k best entries over the sorted lists of all threads of the block, written to out[0..k) (shared or
// global) by warp 0: every warp reduces its lanes' lists to one sorted list, then warp 0 does the same with
// the warps' lists (lane w holds warp w's).  `stage` is shared scratch of kSampleWarps * kMaxTopk candidates.
// Ends with a barrier.
__device__ __forceinline__ void block_topk(const TopList& mine, int k, Cand* out, Cand* stage) {
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

// mix[j] = logsumexp_a(S[a, v + j] + off[a]) for the four vocabulary entries v .. v + 3 (16-byte aligned row
// pieces).  Up to eight experts: all rows are fetched at once and both passes (maximum, sum of exponentials)
// run from registers; more experts: two passes over memory, the second of which hits the caches.
__device__ __forceinline__ void mix_of_four(const float* __restrict__ Srow, int lds, int v, int r,
                                            const float* off_s, float (&mix)[4]) {
  float m[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
  float l[4] = {0.f, 0.f, 0.f, 0.f};
  if (r <= 8) {
    float4 q[8];
#pragma unroll
    for (int a = 0; a < 8; ++a)
      if (a < r) q[a] = __ldg(reinterpret_cast<const float4*>(Srow + static_cast<size_t>(a) * lds + v));
#pragma unroll
    for (int a = 0; a < 8; ++a)
      if (a < r) {
        const float off = off_s[a];
        q[a].x += off; q[a].y += off; q[a].z += off; q[a].w += off;
        m[0] = fmaxf(m[0], q[a].x); m[1] = fmaxf(m[1], q[a].y);
        m[2] = fmaxf(m[2], q[a].z); m[3] = fmaxf(m[3], q[a].w);
      }
#pragma unroll
    for (int a = 0; a < 8; ++a)
      if (a < r) {
        l[0] += __expf(q[a].x - m[0]); l[1] += __expf(q[a].y - m[1]);
        l[2] += __expf(q[a].z - m[2]); l[3] += __expf(q[a].w - m[3]);
      }
  } else {
#pragma unroll 4
    for (int a = 0; a < r; ++a) {
      const float4 q = __ldg(reinterpret_cast<const float4*>(Srow + static_cast<size_t>(a) * lds + v));
      const float off = off_s[a];
      m[0] = fmaxf(m[0], q.x + off); m[1] = fmaxf(m[1], q.y + off);
      m[2] = fmaxf(m[2], q.z + off); m[3] = fmaxf(m[3], q.w + off);
    }
#pragma unroll 4
    for (int a = 0; a < r; ++a) {
      const float4 q = __ldg(reinterpret_cast<const float4*>(Srow + static_cast<size_t>(a) * lds + v));
      const float off = off_s[a];
      l[0] += __expf(q.x + off - m[0]); l[1] += __expf(q.y + off - m[1]);
      l[2] += __expf(q.z + off - m[2]); l[3] += __expf(q.w + off - m[3]);
    }
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) mix[j] = m[j] + __logf(l[j]);
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
      const uint4 e = __ldg(erow + g);
      const float e0 = ptx::bf16_lo(e.x), e1 = ptx::bf16_hi(e.x), e2 = ptx::bf16_lo(e.y), e3 = ptx::bf16_hi(e.y);
      const float e4 = ptx::bf16_lo(e.z), e5 = ptx::bf16_hi(e.z), e6 = ptx::bf16_lo(e.w), e7 = ptx::bf16_hi(e.w);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (a0 + u < r) {
          const float4* zrow = reinterpret_cast<const float4*>(z32 + (row0 + a0 + u) * d);
          const float4 z0 = __ldg(zrow + 2 * g), z1 = __ldg(zrow + 2 * g + 1);
          float t = acc[u];
          t = fmaf(e0, z0.x, t); t = fmaf(e1, z0.y, t); t = fmaf(e2, z0.z, t); t = fmaf(e3, z0.w, t);
          t = fmaf(e4, z1.x, t); t = fmaf(e5, z1.y, t); t = fmaf(e6, z1.z, t); t = fmaf(e7, z1.w, t);
          acc[u] = t;
        }
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

// Conditional log-probabilities of the candidates of draft step s at position i (the reported values, from the
// unrounded z):  topk_logp[i, s, j] = logsumexp_a(log b_a + log P^(s)(cand_j | a)) - logsumexp_a log b_a,
// with b the expert weights BEFORE step s.  This block takes candidates j = first, first + stride, ...
__device__ __forceinline__ void candidate_logps(const uint16_t* __restrict__ E, const float* __restrict__ z32,
                                                const float* __restrict__ lse, const float* __restrict__ lb_before,
                                                const int* __restrict__ cand, int i, int s, int d, int V, int n, int r,
                                                int topk, int first, int stride, float* __restrict__ topk_logp,
                                                float* tgt_s, float* red) {
  const size_t row0 = (static_cast<size_t>(i) * n + s) * r;
  for (int j = first; j < topk; j += stride) {
    // a candidate outside the vocabulary would gather from beyond E (checked build: reported, row 0 read instead)
    int tok = cand[j];
    if (!CPMTP_INDEX_OK(tok, 1, V)) tok = 0;
    block_token_logits(E, tok, z32, lse, row0, d, r, tgt_s, red);
    if (threadIdx.x < 32) {
      const int a = threadIdx.x;
      const float b = a < r ? lb_before[static_cast<size_t>(i) * r + a] : -INFINITY;
      const float mb = warp_max(b);
      const float norm = mb + logf(warp_sum(a < r ? expf(b - mb) : 0.f));
      const float x = a < r ? b + tgt_s[a] : -INFINITY;
      const float m = warp_max(x);
      const float tot = warp_sum(a < r ? expf(x - m) : 0.f);
      if (a == 0) topk_logp[(static_cast<size_t>(i) * n + s) * topk + j] = m + logf(tot) - norm;
    }
    __syncthreads();   // tgt_s and red are reused by the next candidate
  }
}

// One draft step.  Grid (chunks, N), kSampleThreads threads, lb_hist = [n + 1][N][r] (expert weights before
// every step), cand_hist = [n][N][kMaxTopk] (candidate tokens of every step).
//   phase 1 (every block): scan the chunk's entries of position i, mix[v] = logsumexp_a(log b_a + S[s,a,v] - lse[s,a]);
//            keep the k best tokens and, when sampling, the best Gumbel-perturbed score; write them to part_*.
//   phase 2 (the block that raises done[i] to the chunk count, i.e. the last to finish for position i): merge the
//            chunks, choose the token, recompute the chosen token's logits from the unrounded z (fp32; only the
//            *selection* sees bf16-rounded z), fold them into log b for the next step, and reset done[i].
//   side job (blocks with chunk < topk, after their own part): the exact conditional log-probabilities of the
//            candidates of the PREVIOUS step, which nothing later depends on; draft_tail_kernel does the same for
//            the last step.
// No block waits for another: whichever finishes last does the merge.
__global__ void __launch_bounds__(kSampleThreads, kSampleBlocksPerSm)
draft_step_kernel(const float* __restrict__ S, int lds, const float* __restrict__ z32, const uint16_t* __restrict__ E,
                  int d, const float* __restrict__ lse, float* __restrict__ lb_hist, const float* __restrict__ uniform,
                  float inv_temp, int s, int N, int V, int n, int r, int topk, const int32_t* __restrict__ forced,
                  Cand* __restrict__ part_top, Cand* __restrict__ part_best, unsigned int* __restrict__ done,
                  int* __restrict__ cand_hist, int* __restrict__ dev_status, int32_t* __restrict__ draft,
                  float* __restrict__ logp_joint, int32_t* __restrict__ topk_tokens, float* __restrict__ topk_logp) {
  __shared__ float off_s[CPMTP_MAX_R];
  __shared__ float lb_s[CPMTP_MAX_R];
  __shared__ float tgt_s[CPMTP_MAX_R];                  // log P^(s)(token | expert)
  __shared__ float red_f[kSampleWarps * CPMTP_MAX_R];
  __shared__ float norm_s;
  __shared__ Cand red[kSampleWarps];
  __shared__ Cand stage[kSampleWarps * kMaxTopk];
  __shared__ Cand final_top[kMaxTopk];
  __shared__ int tok_s;
  __shared__ bool is_last;
  const int chunk = blockIdx.x, chunks = gridDim.x, i = blockIdx.y;
  const int K = n * r;
  const float* lb = lb_hist + static_cast<size_t>(s) * N * r;              // before this step
  float* lb_next = lb_hist + static_cast<size_t>(s + 1) * N * r;           // after it
  if (threadIdx.x < 32) {
    const int a = threadIdx.x;
    const float b = a < r ? lb[static_cast<size_t>(i) * r + a] : -INFINITY;
    if (a < r) {
      lb_s[a] = b;
      off_s[a] = b - lse[static_cast<size_t>(i) * K + s * r + a];
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
    const float* Srow = S + (static_cast<size_t>(i) * K + static_cast<size_t>(s) * r) * lds;
    const float* urow = uniform != nullptr ? uniform + (static_cast<size_t>(i) * n + s) * V : nullptr;
    TopList top;
    top.init();
    Cand best{-INFINITY, kNoToken};
    const int v_end = min(V, (chunk + 1) * kSampleChunk);
    // two groups of four consecutive vocabulary entries per thread, half a chunk apart (lds % 32 == 0: 16-byte
    // aligned loads, a warp reads 512 contiguous bytes of every row; entries in [V, lds) exist in the buffer
    // and are left out below)
#pragma unroll
    for (int grp = 0; grp < 2; ++grp) {
      const int v0 = chunk * kSampleChunk + grp * (kSampleChunk / 2) + 4 * threadIdx.x;
      if (v0 >= v_end) continue;
      float mix[4];
      mix_of_four(Srow, lds, v0, r, off_s, mix);
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
    top.sort();
    block_topk(top, topk, part_top + (static_cast<size_t>(i) * chunks + chunk) * kMaxTopk, stage);
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
    // ---- phase 2: merge (thread t holds the sorted lists of chunks t, t + 256, ...), choose, fold
    TopList top;
    top.init();
    Cand best{-INFINITY, kNoToken};
    for (int c = threadIdx.x; c < chunks; c += kSampleThreads) {
      const Cand* src = part_top + (static_cast<size_t>(i) * chunks + c) * kMaxTopk;
      for (int j = 0; j < topk; ++j) {
        const Cand pt = load_cand_cg(src + j);
        if (pt.idx != kNoToken) top.insert(pt.score, pt.idx, topk);
      }
      if (uniform != nullptr) {
        const Cand pb = load_cand_cg(part_best + static_cast<size_t>(i) * chunks + c);
        if (cand_better(pb.score, pb.idx, best.score, best.idx)) best = pb;
      }
    }
    block_topk(top, topk, final_top, stage);
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
      done[i] = 0u;   // ready for the next step (launches on the stream are ordered)
    }
    if (threadIdx.x < topk) {
      const int t = final_top[threadIdx.x].idx;
      cand_hist[(static_cast<size_t>(s) * N + i) * kMaxTopk + threadIdx.x] = t;
      if (topk_tokens != nullptr) topk_tokens[(static_cast<size_t>(i) * n + s) * topk + threadIdx.x] = t;
    }
    __syncthreads();
    block_token_logits(E, tok_s, z32, lse, (static_cast<size_t>(i) * n + s) * r, d, r, tgt_s, red_f);
    if (threadIdx.x < 32) {
      const int a = threadIdx.x;
      float bb = -INFINITY;
      if (a < r) {
        bb = lb_s[a] + tgt_s[a];
        lb_next[static_cast<size_t>(i) * r + a] = bb;
      }
      if (s == n - 1 && logp_joint != nullptr) {
        const float m = warp_max(bb);
        const float e = a < r ? expf(bb - m) : 0.f;
        const float tot = warp_sum(e);
        if (a == 0) logp_joint[i] = m + logf(tot);
      }
    }
    __syncthreads();
  }
  // ---- side job: reported log-probabilities of the previous step's candidates
  if (s > 0 && topk_logp != nullptr && chunk < topk) {
    candidate_logps(E, z32, lse, lb_hist + static_cast<size_t>(s - 1) * N * r,
                    cand_hist + (static_cast<size_t>(s - 1) * N + i) * kMaxTopk, i, s - 1, d, V, n, r, topk, chunk,
                    chunks, topk_logp, tgt_s, red_f);
  }
#ifdef CPMTP_DEBUG
  if (threadIdx.x == 0 && dev_status != nullptr) {
    const int seen = *const_cast<volatile int*>(&g_debug_status);
    if (seen != 0) atomicMax(dev_status, seen);
  }
#endif
}

// The candidates' reported log-probabilities for the last draft step.  Grid (topk, N).
__global__ void __launch_bounds__(kSampleThreads, kSampleBlocksPerSm)
draft_tail_kernel(const float* __restrict__ z32, const uint16_t* __restrict__ E, int d, const float* __restrict__ lse,
                  const float* __restrict__ lb_hist, const int* __restrict__ cand_hist, int N, int V, int n, int r,
                  int topk, float* __restrict__ topk_logp) {
  __shared__ float tgt_s[CPMTP_MAX_R];
  __shared__ float red_f[kSampleWarps * CPMTP_MAX_R];
  const int i = blockIdx.y, s = n - 1;
  candidate_logps(E, z32, lse, lb_hist + static_cast<size_t>(s) * N * r,
                  cand_hist + (static_cast<size_t>(s) * N + i) * kMaxTopk, i, s, d, V, n, r, topk, blockIdx.x, gridDim.x,
                  topk_logp, tgt_s, red_f);
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
