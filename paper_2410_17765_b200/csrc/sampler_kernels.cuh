// Draft generation from the factors (sampling section of the paper).
//
// The unembedding GEMM has stored the logits S[(i,k), v] (fp32) and their
// logsumexp; token s of the draft is then chosen from
//   mix[v] = log sum_alpha b_alpha * P^(s)(v | alpha),
//   b_alpha = w_alpha * prod_{t<s} P^(t)(x_t | alpha)          (Eq. 11 for s = 1),
// either greedily or by the Gumbel-max rule on caller-supplied uniforms, and the
// k most likely tokens are reported as candidates for a static draft tree.
// Two small streaming kernels per token: per-chunk partial selection over the
// vocabulary, then a per-position merge that also folds the chosen token's
// factors into b.  Ties go to the lowest token id, so results are reproducible.
#pragma once
#include <cstdint>

#include "../../include/cpmtp.h"
#include "small_kernels.cuh"

namespace cpmtp {

constexpr int kMaxTopk = 8;
constexpr int kSampleThreads = 256;
constexpr int kSampleChunk = 2048;   // vocabulary entries per block in the partial pass
constexpr int kSampleFinalThreads = 1024;   // merge pass: one block per position, one warp per (candidate, expert) dot

struct Cand {
  float score;
  int idx;
};

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
    if (!cand_better(s, i, score[k - 1], idx[k - 1])) return;
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

// Block-wide best candidate (score desc, index asc); result valid in every thread.
__device__ __forceinline__ Cand block_best(Cand c, Cand* red /* [32] shared */) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float os = __shfl_xor_sync(0xffffffffu, c.score, o);
    const int oi = __shfl_xor_sync(0xffffffffu, c.idx, o);
    if (cand_better(os, oi, c.score, c.idx)) {
      c.score = os;
      c.idx = oi;
    }
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  __syncthreads();
  if (lane == 0) red[warp] = c;
  __syncthreads();
  Cand r = lane < nwarps ? red[lane] : Cand{-INFINITY, 0x7fffffff};
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float os = __shfl_xor_sync(0xffffffffu, r.score, o);
    const int oi = __shfl_xor_sync(0xffffffffu, r.idx, o);
    if (cand_better(os, oi, r.score, r.idx)) {
      r.score = os;
      r.idx = oi;
    }
  }
  return r;
}

// Merge the threads' sorted lists into the block's k best, written to out[0..k) by thread 0.
__device__ __forceinline__ void block_topk(const TopList& mine, int k, Cand* out, Cand* red) {
  int head = 0;
  for (int round = 0; round < k; ++round) {
    Cand c{-INFINITY, 0x7fffffff};
#pragma unroll
    for (int j = 0; j < kMaxTopk; ++j)
      if (j == head) c = Cand{mine.score[j], mine.idx[j]};
    if (head >= k) c = Cand{-INFINITY, 0x7fffffff};
    const Cand w = block_best(c, red);
    if (w.idx == c.idx && w.score == c.score && c.idx != 0x7fffffff) ++head;   // indices are unique: one winner
    if (threadIdx.x == 0) out[round] = w;
  }
}

// Pass 1 of one draft step: grid (chunks, N).  Each block scans its chunk of the vocabulary for
// position i: the k best tokens by mix[v] and the best perturbed score.
__global__ void draft_step_partial_kernel(const float* __restrict__ S, int lds, const float* __restrict__ lse,
                                          const float* __restrict__ lb, const float* __restrict__ uniform,
                                          float inv_temp, int s, int V, int n, int r, int topk,
                                          Cand* __restrict__ part_top, Cand* __restrict__ part_best) {
  __shared__ float off_s[CPMTP_MAX_R];
  __shared__ float norm_s;
  __shared__ Cand red[32];
  const int chunk = blockIdx.x, chunks = gridDim.x, i = blockIdx.y;
  const int K = n * r;
  if (threadIdx.x < 32) {
    const int a = threadIdx.x;
    const float b = a < r ? lb[static_cast<size_t>(i) * r + a] : -INFINITY;
    if (a < r) off_s[a] = b - lse[static_cast<size_t>(i) * K + s * r + a];
    const float m = warp_max(b);
    const float e = a < r ? expf(b - m) : 0.f;
    const float tot = warp_sum(e);
    if (a == 0) norm_s = m + logf(tot);
  }
  __syncthreads();
  const float norm = norm_s;
  const float* Srow = S + (static_cast<size_t>(i) * K + static_cast<size_t>(s) * r) * lds;
  const float* urow = uniform != nullptr ? uniform + (static_cast<size_t>(i) * n + s) * V : nullptr;
  TopList top;
  top.init();
  Cand best{-INFINITY, 0x7fffffff};
  const int v_end = min(V, (chunk + 1) * kSampleChunk);
  // four consecutive vocabulary entries per thread and pass (lds % 32 == 0: 16-byte aligned loads; entries in
  // [V, lds) exist in the buffer and are skipped below)
  for (int v0 = chunk * kSampleChunk + 4 * threadIdx.x; v0 < v_end; v0 += 4 * blockDim.x) {
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
  block_topk(top, topk, part_top + (static_cast<size_t>(i) * chunks + chunk) * kMaxTopk, red);
  const Cand b = block_best(best, red);
  if (threadIdx.x == 0) part_best[static_cast<size_t>(i) * chunks + chunk] = b;
}

// Pass 2: one block per position.  Merge the chunks' partial results, emit the token and the
// candidates, fold the chosen token's factors into b, and after the last token the joint log-probability.
// The logits of the drafted token and of the candidates are recomputed from the unrounded z (fp32),
// as on the likelihood path, so the reported log-probabilities do not carry the bf16 rounding of z
// (the selection itself is made on the stored logits; candidates keep the selection order).
__global__ void __launch_bounds__(kSampleFinalThreads) draft_step_final_kernel(const float* __restrict__ z32, const uint16_t* __restrict__ E, int d,
                                        const float* __restrict__ lse,
                                        float* __restrict__ lb, const Cand* __restrict__ part_top,
                                        const Cand* __restrict__ part_best, int chunks, int sampled, int s, int V,
                                        int n, int r, int topk, const int32_t* __restrict__ forced,
                                        int* __restrict__ dev_status, int32_t* __restrict__ draft,
                                        float* __restrict__ logp_joint, int32_t* __restrict__ topk_tokens,
                                        float* __restrict__ topk_logp) {
  __shared__ Cand red[32];
  __shared__ Cand final_top[kMaxTopk];
  __shared__ int cand_tok[kMaxTopk + 1];
  __shared__ float tgt_s[kMaxTopk + 1][CPMTP_MAX_R];   // log P^(s)(candidate | expert)
  __shared__ float norm_s;
  const int i = blockIdx.x;
  const int K = n * r;
  TopList top;
  top.init();
  Cand best{-INFINITY, 0x7fffffff};
  for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
    const Cand* pt = part_top + (static_cast<size_t>(i) * chunks + c) * kMaxTopk;
    for (int j = 0; j < topk; ++j) top.insert(pt[j].score, pt[j].idx, topk);
    const Cand pb = part_best[static_cast<size_t>(i) * chunks + c];
    if (cand_better(pb.score, pb.idx, best.score, best.idx)) best = pb;
  }
  block_topk(top, topk, final_top, red);
  const Cand b = block_best(best, red);
  // log sum_alpha b_alpha before this token is folded in
  if (threadIdx.x < 32) {
    const int a = threadIdx.x;
    const float bb = a < r ? lb[static_cast<size_t>(i) * r + a] : -INFINITY;
    const float m = warp_max(bb);
    const float e = a < r ? expf(bb - m) : 0.f;
    const float tot = warp_sum(e);
    if (a == 0) norm_s = m + logf(tot);
  }
  if (threadIdx.x == 0) {   // the drafted token: the caller's, if one is given for this step
    int tok = sampled ? b.idx : final_top[0].idx;
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
  // Exact logits (from the unrounded z) of the candidates and of the drafted token, for every expert.
  {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    for (int job = warp; job < (topk + 1) * r; job += nwarps) {
      const int j = job / r, a = job - j * r;
      // d % 64 == 0 and 16-byte aligned rows: 8 elements per lane and load
      const uint4* erow = reinterpret_cast<const uint4*>(E + static_cast<size_t>(cand_tok[j]) * d);
      const float4* zrow =
          reinterpret_cast<const float4*>(z32 + (static_cast<size_t>(i) * K + static_cast<size_t>(s) * r + a) * d);
      float acc = 0.f;
      for (int t = lane; t < (d >> 3); t += 32) {
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
      acc = warp_sum(acc);
      if (lane == 0) tgt_s[j][a] = acc - lse[static_cast<size_t>(i) * K + static_cast<size_t>(s) * r + a];
    }
  }
  __syncthreads();
  // conditional log-probabilities of the candidates: logsumexp_a(log b_a + log P^(s)(tok | a)) - norm
  {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    for (int j = warp; j < topk; j += nwarps) {
      const float x = lane < r ? lb[static_cast<size_t>(i) * r + lane] + tgt_s[j][lane] : -INFINITY;
      const float m = warp_max(x);
      const float e = lane < r ? expf(x - m) : 0.f;
      const float tot = warp_sum(e);
      if (lane == 0) {
        if (topk_tokens != nullptr) topk_tokens[(static_cast<size_t>(i) * n + s) * topk + j] = cand_tok[j];
        if (topk_logp != nullptr) topk_logp[(static_cast<size_t>(i) * n + s) * topk + j] = m + logf(tot) - norm_s;
      }
    }
  }
  if (threadIdx.x == 0) draft[static_cast<size_t>(i) * n + s] = cand_tok[topk];
  __syncthreads();
  if (threadIdx.x < 32) {
    const int a = threadIdx.x;
    float bb = -INFINITY;
    if (a < r) {
      bb = lb[static_cast<size_t>(i) * r + a] + tgt_s[topk][a];
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
