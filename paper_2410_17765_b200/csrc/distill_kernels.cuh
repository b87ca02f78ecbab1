// Small stages of the distillation objective (Eq. 14) around its two GEMM passes.
// Reductions run in a fixed order (no floating-point atomics).
#pragma once
#include <cstdint>

#include "../../include/cpmtp.h"
#include "small_kernels.cuh"

namespace cpmtp {

__device__ __forceinline__ float bf16_at(const uint16_t* p, size_t i) {
  return __uint_as_float(static_cast<uint32_t>(__ldg(p + i)) << 16);
}

// log pi[i, s, a]: the expert weights before token s, pi proportional to w_a prod_{t<s} P^(t)(x_t | a)
// (sampling section, teacher-forced on the sequence's own tokens).  One thread per position.
__global__ void distill_pi_kernel(const float* __restrict__ logw, const float* __restrict__ lse,
                                  const float* __restrict__ tgt, float* __restrict__ logpi, int N, int n, int r) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  const int K = n * r;
  float a[CPMTP_MAX_R];
  for (int b = 0; b < r; ++b) a[b] = logw[static_cast<size_t>(i) * r + b];
  for (int s = 0; s < n; ++s) {
    float m = -INFINITY;
    for (int b = 0; b < r; ++b) m = fmaxf(m, a[b]);
    float tot = 0.f;
    for (int b = 0; b < r; ++b) tot += expf(a[b] - m);
    const float norm = m + logf(tot);
    for (int b = 0; b < r; ++b) {
      const size_t row = static_cast<size_t>(i) * K + s * r + b;
      logpi[row] = a[b] - norm;
      a[b] += tgt[row] - lse[row];
    }
  }
}

// One warp per group g = (position, token).  The teacher's normaliser from the sweep's per-split statistics,
//   lse_t[g] = logsumexp_v T[g, v]  (two-pass merge of (max, sum-exp) in the log2 domain),
// then  pm[row] = sum over splits of the pm' partials + pi[row] * lse_t[g]  and  kl[g] = sum_a pm[(g, a)].
__global__ void distill_merge_kernel(const float* __restrict__ part, const float* __restrict__ part_tm,
                                     const float* __restrict__ part_tl, const float* __restrict__ logpi, int splits,
                                     float* __restrict__ lse_t, float* __restrict__ pm, float* __restrict__ kl,
                                     int groups, int r) {
  const int g = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (g >= groups) return;
  float m = -INFINITY;
  for (int j = lane; j < splits; j += 32) m = fmaxf(m, part_tm[static_cast<size_t>(g) * splits + j]);
  m = warp_max(m);
  float l = 0.f;
  for (int j = lane; j < splits; j += 32) {
    const float lj = part_tl[static_cast<size_t>(g) * splits + j];
    if (lj > 0.f) l += lj * exp2f(part_tm[static_cast<size_t>(g) * splits + j] - m);
  }
  l = warp_sum(l);
  const float lt = (m + log2f(l)) * 0.6931471805599453f;
  if (lane == 0) lse_t[g] = lt;
  float total = 0.f;
  for (int a = 0; a < r; ++a) {
    const size_t row = static_cast<size_t>(g) * r + a;
    float v = 0.f;
    for (int j = lane; j < splits; j += 32) v += part[row * splits + j];
    v = warp_sum(v) + expf(logpi[row]) * lt;
    if (lane == 0) pm[row] = v;
    total += v;
  }
  if (lane == 0) kl[g] = total;
}

// Default upstream weights of the loss after Eq. 14, (1/N) sum_i sum_k gamma^k (beta KL_k + (1 - beta) CE_k)
// with CE_k = prefix_{k-1} - prefix_k:  weight of kl[i, k] and of prefix[i, k].
__device__ __forceinline__ float distill_uk(int k, float beta, float gamma, int N) {
  return beta * powf(gamma, static_cast<float>(k)) / N;
}
__device__ __forceinline__ float distill_up(int k, int n, float beta, float gamma, int N) {
  const float gk = powf(gamma, static_cast<float>(k));
  const float next = k + 1 < n ? gk * gamma : 0.f;
  return (1.f - beta) * (next - gk) / N;
}

// loss = sum_i sum_k (up prefix + uk kl) + aux_coef sum_a wbar_a^2, double accumulation, one block.
constexpr int kDistillLossThreads = 512;
__global__ void __launch_bounds__(kDistillLossThreads) distill_loss_kernel(
    const float* __restrict__ prefix, const float* __restrict__ kl, const float* __restrict__ wbar,
    const float* __restrict__ up, const float* __restrict__ uk, float beta, float gamma, float aux_coef, int N, int n,
    int r, float* __restrict__ loss) {
  __shared__ double red[kDistillLossThreads / 32];
  const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
  double acc = 0.0;
  const long long total = static_cast<long long>(N) * n;
  for (long long idx = t; idx < total; idx += kDistillLossThreads) {
    const int k = static_cast<int>(idx % n);
    const float wp = up != nullptr ? up[idx] : distill_up(k, n, beta, gamma, N);
    const float wk = uk != nullptr ? uk[idx] : distill_uk(k, beta, gamma, N);
    acc += static_cast<double>(wp) * prefix[idx] + static_cast<double>(wk) * kl[idx];
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) red[warp] = acc;
  __syncthreads();
  if (t == 0) {
    double v = 0.0;
    for (int w = 0; w < kDistillLossThreads / 32; ++w) v += red[w];
    double aux = 0.0;
    for (int b = 0; b < r; ++b) aux += static_cast<double>(wbar[b]) * wbar[b];
    *loss = static_cast<float>(v + static_cast<double>(aux_coef) * aux);
  }
}

// Backward coefficients of  sum up * prefix + sum uk * kl (+ the balance term), one thread per position.
// Cross-entropy path as in coeff_kernel's per-token form.  KL path: with b the unnormalised expert
// weights before token k,  d kl_k / d log b_{k,a} = pm_{k,a} - pi_{k,a} kl_k =: tb_{k,a} / uk_k, and
// log b_{k,a} = log w_a + sum_{t<k} C[t,a], so tb_k joins the coefficients of every earlier head and the
// gate.  Also writes the kl weights actually used, uk_out[i, k].
__global__ void distill_coeff_kernel(const float* __restrict__ logw, const float* __restrict__ wbar,
                                     const float* __restrict__ lse, const float* __restrict__ tgt,
                                     const float* __restrict__ logpi, const float* __restrict__ pm,
                                     const float* __restrict__ kl, const float* __restrict__ up,
                                     const float* __restrict__ uk, float beta, float gamma, float* __restrict__ coef,
                                     float* __restrict__ dg, float* __restrict__ uk_out, int N, int n, int r,
                                     float aux_coef) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  const int K = n * r;
  const float scale = 2.0f * aux_coef / N;
  float wu = 0.f;
  for (int b = 0; b < r; ++b) wu += expf(logw[static_cast<size_t>(i) * r + b]) * scale * wbar[b];
  float a[CPMTP_MAX_R], acc[CPMTP_MAX_R], D[CPMTP_MAX_R];
  float up_sum = 0.f;
  for (int b = 0; b < r; ++b) {
    a[b] = logw[static_cast<size_t>(i) * r + b];
    acc[b] = 0.f;
  }
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
    const size_t g = static_cast<size_t>(i) * n + s;
    const float u_s = up != nullptr ? up[g] : distill_up(s, n, beta, gamma, N);
    uk_out[g] = uk != nullptr ? uk[g] : distill_uk(s, beta, gamma, N);
    up_sum += u_s;
    for (int b = 0; b < r; ++b) {
      const float wq = u_s * expf(a[b] - m) * inv;
      coef[static_cast<size_t>(i) * K + s * r + b] = wq;
      acc[b] += wq;
    }
  }
  float d_sum = 0.f;
  for (int b = 0; b < r; ++b) {
    float run = 0.f, later = 0.f;   // later = sum_{k > s} tb[k, b]
    for (int s = n - 1; s >= 0; --s) {
      const size_t row = static_cast<size_t>(i) * K + s * r + b;
      run += coef[row];
      coef[row] = run + later;
      later += uk_out[static_cast<size_t>(i) * n + s] * (pm[row] - expf(logpi[row]) * kl[static_cast<size_t>(i) * n + s]);
    }
    D[b] = later;
    d_sum += later;
  }
  for (int b = 0; b < r; ++b) {
    const float w = expf(logw[static_cast<size_t>(i) * r + b]);
    dg[static_cast<size_t>(i) * r + b] = acc[b] - up_sum * w + D[b] - w * d_sum + w * (scale * wbar[b] - wu);
  }
}

}  // namespace cpmtp
