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
// memory, no waiting anywhere) merges the chunks, folds the chosen token's factors into b and
// writes the step's outputs.  Ties go to the lowest token id, so results are reproducible.
#pragma once
#include <cstdint>

#include "../../include/cpmtp.h"
#include "small_kernels.cuh"
#include "tc_gemm.cuh"

namespace cpmtp {

constexpr int kMaxTopk = 8;
constexpr int kSampleThreads = 1024;
constexpr int kSampleChunk = 4096;   // vocabulary entries per block: four per thread

struct __align__(8) Cand {
  float score;
  int idx;
};

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
      idx[j] = 0x7fffffff;
    }
  }
  __device__ void insert(float s, int i, int k) {
    float last_s = -INFINITY;
    int last_i = 0x7fffffff;
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
__device__ __forceinline__ Cand block_best(Cand c, Cand* red /* [32] shared */) {
  c = warp_best(c);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  __syncthreads();
  if (lane == 0) red[warp] = c;
  __syncthreads();
  return warp_best(lane < nwarps ? red[lane] : Cand{-INFINITY, 0x7fffffff});
}

// The k best entries over the sorted lists of a warp's lanes (token ids are unique, so every round
// has one winner): lane t < k returns the t-th best, the other lanes an empty candidate.
__device__ __forceinline__ Cand warp_topk(const TopList& mine, int k) {
  const int lane = threadIdx.x & 31;
  int head = 0;
  Cand res{-INFINITY, 0x7fffffff};
  for (int round = 0; round < k; ++round) {
    Cand c{-INFINITY, 0x7fffffff};
#pragma unroll
    for (int j = 0; j < kMaxTopk; ++j)
      if (j == head && j < k) c = Cand{mine.score[j], mine.idx[j]};
    const Cand w = warp_best(c);
    if (w.idx == c.idx && c.idx != 0x7fffffff) ++head;
    if (lane == round) res = w;
  }
  return res;
}

// The k best entries over the lists of all threads of the block, written to out[0..k) (shared or
// global) by warp 0; `stage` is shared scratch of 32 * kMaxTopk candidates.  Ends with a barrier.
__device__ __forceinline__ void block_topk(const TopList& mine, int k, Cand* out, Cand* stage) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const Cand w = warp_topk(mine, k);
  __syncthreads();   // `stage` may still be read from a previous use
  if (lane < k) stage[warp * kMaxTopk + lane] = w;
  __syncthreads();
  if (warp == 0) {
    TopList merged;
    merged.init();
    for (int e = lane; e < nwarps * kMaxTopk; e += 32) {
      const int wsrc = e / kMaxTopk, j = e - wsrc * kMaxTopk;
      if (j < k) {
        const Cand c = stage[wsrc * kMaxTopk + j];
        if (c.idx != 0x7fffffff) merged.insert(c.score, c.idx, k);
      }
    }
    const Cand f = warp_topk(merged, k);
    if (lane < k) out[lane] = f;
  }
  __syncthreads();
}

// fp32 z row (8 elements per step) against a bf16 row of E over [lo, hi) steps of 8 elements with stride `step`.
__device__ __forceinline__ float dot_e_z(const uint4* __restrict__ erow, const float4* __restrict__ zrow, int lo,
                                         int hi, int step) {
  float acc = 0.f;
#pragma unroll 4
  for (int t = lo; t < hi; t += step) {
    const uint4 e = __ldg(erow + t);
    const float4 z0 = zrow[2 * t], z1 = zrow[2 * t + 1];
    acc = fmaf(ptx::bf16_lo(e.x), z0.x, acc);
    acc = fmaf(ptx::bf16_hi(e.x), z0.y, acc);
    acc = fmaf(ptx::bf16_lo(e.y), z0.z, acc);
    acc = fmaf(ptx::bf16_hi(e.y), z0.w, acc);
    acc = fmaf(ptx::bf16_lo(e.z), z1.x, acc);
    acc = fmaf(ptx::bf16_hi(e.z), z1.y, acc);
    acc = fmaf(ptx::bf16_lo(e.w), z1.z, acc);
    acc = fmaf(ptx::bf16_hi(e.w), z1.w, acc);
  }
  return acc;
}

// One draft step.  Grid (chunks, N), kSampleThreads threads.
//   phase 1 (every block): scan the chunk's entries of position i, mix[v] = logsumexp_a(log b_a + S[s,a,v] - lse[s,a]);
//            keep the k best tokens and, when sampling, the best Gumbel-perturbed score; write them to part_*.
//   phase 2 (the block that raises done[i] to the chunk count, i.e. the last to finish for position i): merge the
//            chunks, choose the token, recompute the logits of the token and of the candidates from the unrounded
//            z (fp32; only the *selection* sees bf16-rounded z), emit the outputs, fold the token's factors into
//            log b, and reset done[i] for the next step.
// No block waits for another: whichever finishes last does the merge.
__global__ void __launch_bounds__(kSampleThreads)
draft_step_kernel(const float* __restrict__ S, int lds, const float* __restrict__ z32, const uint16_t* __restrict__ E,
                  int d, const float* __restrict__ lse, float* __restrict__ lb, const float* __restrict__ uniform,
                  float inv_temp, int s, int V, int n, int r, int topk, const int32_t* __restrict__ forced,
                  Cand* __restrict__ part_top, Cand* __restrict__ part_best, unsigned int* __restrict__ done,
                  int* __restrict__ dev_status, int32_t* __restrict__ draft, float* __restrict__ logp_joint,
                  int32_t* __restrict__ topk_tokens, float* __restrict__ topk_logp) {
  __shared__ float off_s[CPMTP_MAX_R];
  __shared__ float lb_s[CPMTP_MAX_R];
  __shared__ float norm_s;
  __shared__ Cand red[32];
  __shared__ Cand stage[32 * kMaxTopk];
  __shared__ Cand final_top[kMaxTopk];
  __shared__ int cand_tok[kMaxTopk + 1];
  __shared__ float tgt_s[kMaxTopk + 1][CPMTP_MAX_R];   // log P^(s)(candidate | expert)
  __shared__ bool is_last;
  const int chunk = blockIdx.x, chunks = gridDim.x, i = blockIdx.y;
  const int K = n * r;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
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
    Cand best{-INFINITY, 0x7fffffff};
    const int v_end = min(V, (chunk + 1) * kSampleChunk);
    // four consecutive vocabulary entries per thread (lds % 32 == 0: 16-byte aligned loads; entries in [V, lds)
    // exist in the buffer and are skipped below)
    const int v0 = chunk * kSampleChunk + 4 * threadIdx.x;
    if (v0 < v_end) {
      // two passes over the r logits (the second one hits L1): maximum first, then the sum of exponentials
      float m[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll 4
      for (int a = 0; a < r; ++a) {
        const float4 q = *reinterpret_cast<const float4*>(Srow + static_cast<size_t>(a) * lds + v0);
        const float off = off_s[a];
        m[0] = fmaxf(m[0], q.x + off); m[1] = fmaxf(m[1], q.y + off);
        m[2] = fmaxf(m[2], q.z + off); m[3] = fmaxf(m[3], q.w + off);
      }
      float l[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
      for (int a = 0; a < r; ++a) {
        const float4 q = *reinterpret_cast<const float4*>(Srow + static_cast<size_t>(a) * lds + v0);
        const float off = off_s[a];
        l[0] += __expf(q.x + off - m[0]); l[1] += __expf(q.y + off - m[1]);
        l[2] += __expf(q.z + off - m[2]); l[3] += __expf(q.w + off - m[3]);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int v = v0 + j;
        if (v >= v_end) continue;
        const float mix = m[j] + __logf(l[j]);
        top.insert(mix, v, topk);
        float sc = mix;
        if (urow != nullptr) sc = (mix - norm) * inv_temp - logf(-logf(urow[v]));
        if (cand_better(sc, v, best.score, best.idx)) best = Cand{sc, v};
      }
    }
    block_topk(top, topk, part_top + (static_cast<size_t>(i) * chunks + chunk) * kMaxTopk, stage);
    const Cand b = block_best(best, red);
    if (threadIdx.x == 0) part_best[static_cast<size_t>(i) * chunks + chunk] = b;
  }
  // ---- who is last for this position?
  __threadfence();   // this block's partial results are visible device-wide before the counter moves
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int prev = atomicAdd(done + i, 1u);
    is_last = prev + 1u == static_cast<unsigned int>(chunks);
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();   // the other blocks' partial results, published before their increments, are read below
  // ---- phase 2: merge, choose, emit
  TopList top;
  top.init();
  Cand best{-INFINITY, 0x7fffffff};
  for (int e = threadIdx.x; e < chunks * topk; e += blockDim.x) {
    const int c = e / topk, j = e - c * topk;
    const Cand pt = load_cand_cg(part_top + (static_cast<size_t>(i) * chunks + c) * kMaxTopk + j);
    if (pt.idx != 0x7fffffff) top.insert(pt.score, pt.idx, topk);
  }
  for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
    const Cand pb = load_cand_cg(part_best + static_cast<size_t>(i) * chunks + c);
    if (cand_better(pb.score, pb.idx, best.score, best.idx)) best = pb;
  }
  block_topk(top, topk, final_top, stage);
  const Cand b = block_best(best, red);
  if (threadIdx.x == 0) {   // the drafted token: the caller's, if one is given for this step
    int tok = uniform != nullptr ? b.idx : final_top[0].idx;
    if (forced != nullptr) {
      const int f = forced[static_cast<size_t>(i) * n + s];
      if (f >= V) {
        if (dev_status != nullptr) atomicMax(dev_status, 1);   // out of range: clamped and reported
        tok = V - 1;
      } else if (f >= 0) {
        tok = f;
      }
    }
    cand_tok[topk] = tok;
  }
  if (threadIdx.x < topk) cand_tok[threadIdx.x] = final_top[threadIdx.x].idx;
  __syncthreads();
  // Exact logits (from the unrounded z) of the candidates and of the drafted token, for every expert:
  // one half-warp per (token, expert) pair; d % 64 == 0 and 16-byte aligned rows.
  {
    const int jobs = (topk + 1) * r;
    const int l16 = lane & 15;
    for (int base = warp * 2; base < jobs; base += 2 * (blockDim.x >> 5)) {
      const int job = base + (lane >> 4);
      const bool active = job < jobs;
      const int jj = active ? job : 0;
      const int j = jj / r, a = jj - j * r;
      // a candidate outside the vocabulary would gather from beyond E (checked build: reported, row 0 read instead)
      const int tok_j = CPMTP_INDEX_OK(cand_tok[j], 1, V) ? cand_tok[j] : 0;
      const uint4* erow = reinterpret_cast<const uint4*>(E + static_cast<size_t>(tok_j) * d);
      const float4* zrow =
          reinterpret_cast<const float4*>(z32 + (static_cast<size_t>(i) * K + static_cast<size_t>(s) * r + a) * d);
      float acc = dot_e_z(erow, zrow, l16, d >> 3, 16);
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      if (active && l16 == 0) tgt_s[j][a] = acc - lse[static_cast<size_t>(i) * K + static_cast<size_t>(s) * r + a];
    }
  }
  __syncthreads();
  // conditional log-probabilities of the candidates: logsumexp_a(log b_a + log P^(s)(tok | a)) - norm
  for (int j = warp; j < topk; j += blockDim.x >> 5) {
    const float x = lane < r ? lb_s[lane] + tgt_s[j][lane] : -INFINITY;
    const float m = warp_max(x);
    const float e = lane < r ? expf(x - m) : 0.f;
    const float tot = warp_sum(e);
    if (lane == 0) {
      if (topk_tokens != nullptr) topk_tokens[(static_cast<size_t>(i) * n + s) * topk + j] = cand_tok[j];
      if (topk_logp != nullptr) topk_logp[(static_cast<size_t>(i) * n + s) * topk + j] = m + logf(tot) - norm;
    }
  }
  if (threadIdx.x == 0) {
    draft[static_cast<size_t>(i) * n + s] = cand_tok[topk];
    done[i] = 0u;   // ready for the next step (launches on the stream are ordered)
#ifdef CPMTP_DEBUG
    const int seen = *const_cast<volatile int*>(&g_debug_status);
    if (seen != 0 && dev_status != nullptr) atomicMax(dev_status, seen);
#endif
  }
  if (threadIdx.x < 32) {
    const int a = threadIdx.x;
    float bb = -INFINITY;
    if (a < r) {
      bb = lb_s[a] + tgt_s[topk][a];
      lb[static_cast<size_t>(i) * r + a] = bb;
    }
    if (s == n - 1 && logp_joint != nullptr) {
      const float m = warp_max(bb);
      const float e = a < r ? expf(bb - m) : 0.f;
      const float tot = warp_sum(e);
      if (a == 0) logp_joint[i] = m + logf(tot);
    }
  }
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
