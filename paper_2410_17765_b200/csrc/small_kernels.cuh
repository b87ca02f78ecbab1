// The O(N*r) and O(N*r*d) stages around the tensor-core GEMMs: gate, mixture
// epilogue, loss, backward coefficients, gate-weight gradient, dtype conversion.
// All reductions run in a fixed order (no floating-point atomics) so results are
// reproducible from run to run.
#pragma once
#include <cstdint>

#include "../../include/cpmtp.h"
#include "ptx.cuh"

namespace cpmtp {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Gate (Eq. 7) and mixture epilogue (last line of Eq. 9) in one launch.  One block
// per position.  Phase 1: warps share the r experts, g[a] = W_g[a] . h[i], then
// logw = log softmax(g).  Phase 2: warps share the n*r heads,
//   lse[i,k]  = two-pass merge of the per-split (max, sum-exp) partials
//   tgt[i,k]  = sum of the per-64-column target-logit partials
// Phase 3 (warp 0, lane = expert):
//   a[i,al]   = logw[i,al] + sum_s (tgt - lse)[i, s*r+al]
//   logp[i]   = logsumexp_al a;  q = exp(a - logp)
// and optionally the prefix scores logsumexp_al(logw + sum_{t<=s} C) for every s.
__global__ void gate_mixture_kernel(const uint16_t* __restrict__ h, const uint16_t* __restrict__ W_g, int d,
                                    const float* __restrict__ part_m, const float* __restrict__ part_l,
                                    int splits, const float* __restrict__ tgt_part, int tgt_parts,
                                    float* __restrict__ logw_out, float* __restrict__ lse_out,
                                    float* __restrict__ tgt_out, float* __restrict__ q_out,
                                    float* __restrict__ logp, float* __restrict__ logp_prefix, int N, int n,
                                    int r) {
  __shared__ float c_s[CPMTP_MAX_N * CPMTP_MAX_R];
  __shared__ float g_s[CPMTP_MAX_R];
  const int i = blockIdx.x;
  const int warp = threadIdx.x >> 5;
  const int nwarps = blockDim.x >> 5;
  const int lane = threadIdx.x & 31;
  const int K = n * r;
  // phase 1: gate logits
  {
    const uint4* hrow = reinterpret_cast<const uint4*>(h + static_cast<size_t>(i) * d);
    const int vecs = d >> 3;
    for (int a = warp; a < r; a += nwarps) {
      const uint4* wrow = reinterpret_cast<const uint4*>(W_g + static_cast<size_t>(a) * d);
      float acc = 0.f;
      for (int j = lane; j < vecs; j += 32) {
        const uint4 hv = __ldg(hrow + j);
        const uint4 wv = __ldg(wrow + j);
        acc = fmaf(ptx::bf16_lo(hv.x), ptx::bf16_lo(wv.x), acc);
        acc = fmaf(ptx::bf16_hi(hv.x), ptx::bf16_hi(wv.x), acc);
        acc = fmaf(ptx::bf16_lo(hv.y), ptx::bf16_lo(wv.y), acc);
        acc = fmaf(ptx::bf16_hi(hv.y), ptx::bf16_hi(wv.y), acc);
        acc = fmaf(ptx::bf16_lo(hv.z), ptx::bf16_lo(wv.z), acc);
        acc = fmaf(ptx::bf16_hi(hv.z), ptx::bf16_hi(wv.z), acc);
        acc = fmaf(ptx::bf16_lo(hv.w), ptx::bf16_lo(wv.w), acc);
        acc = fmaf(ptx::bf16_hi(hv.w), ptx::bf16_hi(wv.w), acc);
      }
      acc = warp_sum(acc);
      if (lane == 0) g_s[a] = acc;
    }
  }
  // The gate above reads only the caller's inputs; the partial results below come from the kernel before
  // this one in the stream (see ptx::grid_dep_wait).
  ptx::grid_dep_wait();
  // phase 2: per-head vocabulary logsumexp and target logit
  for (int k = warp; k < K; k += nwarps) {
    const size_t row = static_cast<size_t>(i) * K + k;
    float m = -INFINITY;
    for (int j = lane; j < splits; j += 32) m = fmaxf(m, part_m[row * splits + j]);
    m = warp_max(m);
    float l = 0.f;
    for (int j = lane; j < splits; j += 32)
      l += part_l[row * splits + j] * exp2f(part_m[row * splits + j] - m);
    l = warp_sum(l);
    const float lse = (m + log2f(l)) * 0.6931471805599453f;
    float t = 0.f;
    for (int j = lane; j < tgt_parts; j += 32) t += tgt_part[row * tgt_parts + j];
    t = warp_sum(t);
    if (lane == 0) {
      c_s[k] = t - lse;
      if (lse_out != nullptr) lse_out[row] = lse;
      if (tgt_out != nullptr) tgt_out[row] = t;
    }
  }
  __syncthreads();
  if (warp != 0) return;
  // phase 3: gate softmax and expert mixture
  float a;
  {
    const float mine = lane < r ? g_s[lane] : -INFINITY;
    const float m = warp_max(mine);
    const float e = lane < r ? expf(mine - m) : 0.f;
    a = mine - (m + logf(warp_sum(e)));
    if (lane < r) logw_out[static_cast<size_t>(i) * r + lane] = a;
  }
  for (int s = 0; s < n; ++s) {
    if (lane < r) a += c_s[s * r + lane];
    if (logp_prefix != nullptr || s == n - 1) {
      const float m = warp_max(a);
      const float e = lane < r ? expf(a - m) : 0.f;
      const float lp = m + logf(warp_sum(e));
      if (logp_prefix != nullptr && lane == 0) logp_prefix[static_cast<size_t>(i) * n + s] = lp;
      if (s == n - 1) {
        if (lane == 0) logp[i] = lp;
        if (q_out != nullptr && lane < r) q_out[static_cast<size_t>(i) * r + lane] = expf(a - lp);
      }
    }
  }
}

// Loss, mean gate weights and hard expert counts (Eq. 10's n_a).  One block, one pass:
//   wbar[a] = (1/N) sum_i exp(logw[i,a]);  counts[a] = #{i : argmax_b w[i,b] = a} (ties -> lowest a)
//   loss = -(1/N) sum_i logp[i] + aux_coef * sum_a wbar[a]^2
// Every thread accumulates its positions in double precision; the per-thread sums are then
// combined in a fixed order (warp shuffles, then across warps), so the result is reproducible.
constexpr int kFinalizeThreads = 512;
__global__ void __launch_bounds__(kFinalizeThreads) finalize_kernel(const float* __restrict__ logp, const float* __restrict__ logw,
                                float* __restrict__ wbar, int* __restrict__ counts,
                                float* __restrict__ loss, int N, int r, float aux_coef) {
  __shared__ double sum_s[32][CPMTP_MAX_R + 1];
  __shared__ int cnt_s[32][CPMTP_MAX_R];
  const int t = threadIdx.x, warp = t >> 5, lane = t & 31, nwarps = blockDim.x >> 5;
  double acc[CPMTP_MAX_R + 1];
  int cnt[CPMTP_MAX_R];
#pragma unroll
  for (int a = 0; a <= CPMTP_MAX_R; ++a) acc[a] = 0.0;
#pragma unroll
  for (int a = 0; a < CPMTP_MAX_R; ++a) cnt[a] = 0;
  for (int i = t; i < N; i += blockDim.x) {
    const float* row = logw + static_cast<size_t>(i) * r;
    float best = -INFINITY;
    int arg = 0;
#pragma unroll
    for (int a = 0; a < CPMTP_MAX_R; ++a) {
      if (a < r) {
        const float v = row[a];
        acc[a] += static_cast<double>(expf(v));
        if (v > best) {
          best = v;
          arg = a;
        }
      }
    }
#pragma unroll
    for (int a = 0; a < CPMTP_MAX_R; ++a) cnt[a] += (a == arg) ? 1 : 0;
    acc[CPMTP_MAX_R] += static_cast<double>(logp[i]);
  }
#pragma unroll
  for (int a = 0; a <= CPMTP_MAX_R; ++a) {
    if (a < r || a == CPMTP_MAX_R) {
      double v = acc[a];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) sum_s[warp][a] = v;
    }
  }
#pragma unroll
  for (int a = 0; a < CPMTP_MAX_R; ++a) {
    if (a < r) {
      int c = cnt[a];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
      if (lane == 0) cnt_s[warp][a] = c;
    }
  }
  __syncthreads();
  if (t <= CPMTP_MAX_R && (t < r || t == CPMTP_MAX_R)) {
    double v = 0.0;
    int c = 0;
    for (int w = 0; w < nwarps; ++w) {
      v += sum_s[w][t];
      if (t < r) c += cnt_s[w][t];
    }
    sum_s[0][t] = v;
    if (t < r) {
      if (wbar != nullptr) wbar[t] = static_cast<float>(v / N);
      if (counts != nullptr) counts[t] = c;
    }
  }
  __syncthreads();
  if (t == 0 && loss != nullptr) {
    double aux = 0.0;
    for (int b2 = 0; b2 < r; ++b2) aux += (sum_s[0][b2] / N) * (sum_s[0][b2] / N);
    *loss = static_cast<float>(-sum_s[0][CPMTP_MAX_R] / N + static_cast<double>(aux_coef) * aux);
  }
}

// Backward coefficients (derivative of Eq. 9 and of the gate softmax of Eq. 7), one thread per position.
//   coef[i, t*r + a] = d objective / d C[i, t, a]        dg[i, b] = d objective / d (W_g h)[i, b]
// Plain objective  sum_i up_i logp_i  (up == nullptr: up_i = -1/N):
//   coef[i, t, a] = up_i q[i, a] for every t;  dg = up_i (q - w) + aux part.
// Per-token objective  sum_i sum_s up[i, s] * log P(x_1..x_{s+1})  (per_token != 0, up is [N, n]):
//   with q_s the expert posterior after s+1 tokens,  coef[i, t, a] = sum_{s >= t} up[i, s] q_s[i, a],
//   dg = sum_s up[i, s] (q_s - w) + aux part.
// aux part (soft balance term): w_b (u_b - sum_g w_g u_g), u_b = 2 aux wbar_b / N.
__global__ void coeff_kernel(const float* __restrict__ q, const float* __restrict__ logw,
                             const float* __restrict__ wbar, const float* __restrict__ lse,
                             const float* __restrict__ tgt, const float* __restrict__ up, int per_token,
                             float* __restrict__ coef, float* __restrict__ dg, int N, int n, int r,
                             float aux_coef) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  const int K = n * r;
  const float scale = 2.0f * aux_coef / N;
  float wu = 0.f;
  for (int b = 0; b < r; ++b) wu += expf(logw[static_cast<size_t>(i) * r + b]) * scale * wbar[b];
  if (!per_token) {
    const float u_i = up != nullptr ? up[i] : -1.0f / N;
    for (int b = 0; b < r; ++b) {
      const float w = expf(logw[static_cast<size_t>(i) * r + b]);
      const float qq = q[static_cast<size_t>(i) * r + b];
      for (int t = 0; t < n; ++t) coef[static_cast<size_t>(i) * K + t * r + b] = u_i * qq;
      dg[static_cast<size_t>(i) * r + b] = u_i * (qq - w) + w * (scale * wbar[b] - wu);
    }
    return;
  }
  float a[CPMTP_MAX_R];
  float acc[CPMTP_MAX_R];   // sum_s up_s q_s[b]
  float up_sum = 0.f;
  for (int b = 0; b < r; ++b) {
    a[b] = logw[static_cast<size_t>(i) * r + b];
    acc[b] = 0.f;
  }
  // forward over s: weighted posteriors, parked in coef[i, s, :]
  for (int s = 0; s < n; ++s) {
    float m = -INFINITY;
    for (int b = 0; b < r; ++b) {
      const size_t row = static_cast<size_t>(i) * K + s * r + b;
      a[b] += tgt[row] - lse[row];
      m = fmaxf(m, a[b]);
    }
    float tot = 0.f;
    for (int b = 0; b < r; ++b) tot += expf(a[b] - m);
    const float inv = 1.0f / tot;
    const float u_s = up[static_cast<size_t>(i) * n + s];
    up_sum += u_s;
    for (int b = 0; b < r; ++b) {
      const float wq = u_s * expf(a[b] - m) * inv;
      coef[static_cast<size_t>(i) * K + s * r + b] = wq;
      acc[b] += wq;
    }
  }
  // suffix sums over s, in place
  for (int b = 0; b < r; ++b) {
    float run = 0.f;
    for (int s = n - 1; s >= 0; --s) {
      run += coef[static_cast<size_t>(i) * K + s * r + b];
      coef[static_cast<size_t>(i) * K + s * r + b] = run;
    }
    const float w = expf(logw[static_cast<size_t>(i) * r + b]);
    dg[static_cast<size_t>(i) * r + b] = acc[b] - up_sum * w + w * (scale * wbar[b] - wu);
  }
}

// dW_g[b, :] = sum_i dg[i, b] * h[i, :]  in two deterministic stages.
// Stage 1: block (column chunk, position slice) -> part[slice, b, col].
template <int R_MAX>
__global__ void dwg_partial_kernel(const float* __restrict__ dg, const uint16_t* __restrict__ h,
                                   float* __restrict__ part, int N, int d, int r, int rows_per_slice) {
  const int col = blockIdx.x * blockDim.x + threadIdx.x;
  const int slice = blockIdx.y;
  if (col >= d) return;
  float acc[R_MAX];
#pragma unroll
  for (int b = 0; b < R_MAX; ++b) acc[b] = 0.f;
  const int i0 = slice * rows_per_slice;
  const int i1 = min(N, i0 + rows_per_slice);
  for (int i = i0; i < i1; ++i) {
    const float hv = __uint_as_float(static_cast<uint32_t>(h[static_cast<size_t>(i) * d + col]) << 16);
    const float* g = dg + static_cast<size_t>(i) * r;
#pragma unroll
    for (int b = 0; b < R_MAX; ++b)
      if (b < r) acc[b] = fmaf(g[b], hv, acc[b]);
  }
#pragma unroll
  for (int b = 0; b < R_MAX; ++b)
    if (b < r) part[(static_cast<size_t>(slice) * r + b) * d + col] = acc[b];
}
// Stage 2: sum the slices in order (on top of the stored value when accumulating) and round to bf16.
__global__ void dwg_reduce_kernel(const float* __restrict__ part, uint16_t* __restrict__ dW_g, int slices,
                                  int r, int d, int accumulate) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= r * d) return;
  float acc = accumulate ? __uint_as_float(static_cast<uint32_t>(dW_g[idx]) << 16) : 0.f;
  for (int s = 0; s < slices; ++s) acc += part[static_cast<size_t>(s) * r * d + idx];
  dW_g[idx] = static_cast<uint16_t>(ptx::pack_bf16x2(acc, 0.f) & 0xFFFFu);
}

// dh[i, :] = bf16( acc[i, :] + sum_b dg[i, b] * W_g[b, :] ): the gate path of Eq. 7 added to an fp32 sum.
__global__ void dh_finish_kernel(const float* __restrict__ acc, const float* __restrict__ dg,
                                 const uint16_t* __restrict__ W_g, uint16_t* __restrict__ dh, int N, int d, int r,
                                 int accumulate) {
  const size_t idx = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= static_cast<size_t>(N) * d) return;
  const int i = static_cast<int>(idx / d), j = static_cast<int>(idx - static_cast<size_t>(i) * d);
  float v = acc[idx];
  if (accumulate) v += __uint_as_float(static_cast<uint32_t>(dh[idx]) << 16);
  for (int b = 0; b < r; ++b)
    v = fmaf(dg[static_cast<size_t>(i) * r + b], __uint_as_float(static_cast<uint32_t>(W_g[static_cast<size_t>(b) * d + j]) << 16), v);
  dh[idx] = static_cast<uint16_t>(ptx::pack_bf16x2(v, 0.f) & 0xFFFFu);
}

// dst = bf16(src), or bf16(src + dst) when accumulating.  count % 4 == 0.
__global__ void f32_to_bf16_kernel(const float* __restrict__ src, uint16_t* __restrict__ dst, size_t count,
                                   int accumulate) {
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x * 4;
  for (size_t i = (static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x) * 4; i < count; i += stride) {
    float4 v = *reinterpret_cast<const float4*>(src + i);
    if (accumulate) {
      const uint2 old = *reinterpret_cast<const uint2*>(dst + i);
      v.x += ptx::bf16_lo(old.x); v.y += ptx::bf16_hi(old.x);
      v.z += ptx::bf16_lo(old.y); v.w += ptx::bf16_hi(old.y);
    }
    uint2 o;
    o.x = ptx::pack_bf16x2(v.x, v.y);
    o.y = ptx::pack_bf16x2(v.z, v.w);
    *reinterpret_cast<uint2*>(dst + i) = o;
  }
}

}  // namespace cpmtp
