// Gaussian-mixture output heads (the paper's appendix on model variants): per token an explicit mixture
// p(x) = sum_k pi_k N(x; mu_k, diag(sigma_k^2)) instead of a diffusion head.  Both densities are closed forms, so a
// round is: draft samples x_i ~ q_i, ratio p_i(x_i) / q_i(x_i), accepted prefix (Sec. 3.1 rule, Alg. 1), and
// acceptance-rejection resampling of the first rejected position from max(0, p - q)/Z (Eq. 5, Eq. 9-11) with
// proposals from p.  One warp per token row, one lane per coordinate (C <= 32); components are walked in order.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace csd {

struct GmmView {
  int K;
  const float* logw;       // [rows, K] unnormalised log-weights
  const float* mu;         // [rows, K, C]
  const float* log_sigma;  // [rows, K, C]
};

// log of the weights' normaliser, log sum_k exp(logw_k); every lane computes the same value
__device__ __forceinline__ float gmm_log_norm(const GmmView& m, size_t row) {
  const float* lw = m.logw + row * m.K;
  float mx = lw[0];
  for (int k = 1; k < m.K; ++k) mx = fmaxf(mx, lw[k]);
  float se = 0.0f;
  for (int k = 0; k < m.K; ++k) se += expf(lw[k] - mx);
  return mx + logf(se);
}

// log-density of the row's mixture at x (lane c < C holds coordinate c); every lane returns it.  The same
// instruction sequence for every mixture, so identical mixtures give identical bits.
__device__ __forceinline__ float gmm_row_logpdf(const GmmView& m, size_t row, int C, int lane, float x) {
  const float lse = gmm_log_norm(m, row);
  float run_m = -INFINITY, run_s = 0.0f;
  for (int k = 0; k < m.K; ++k) {
    float t = 0.0f, sl = 0.0f;
    if (lane < C) {
      const size_t o = (row * m.K + k) * C + lane;
      sl = m.log_sigma[o];
      const float d = (x - m.mu[o]) * expf(-sl);
      t = d * d;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { t += __shfl_xor_sync(0xffffffffu, t, o); sl += __shfl_xor_sync(0xffffffffu, sl, o); }
    const float comp = (m.logw[row * m.K + k] - lse) - sl - 0.5f * t - 0.9189385332046727f * C;   // C/2 log(2 pi)
    if (comp > run_m) { run_s = run_s * expf(run_m - comp) + 1.0f; run_m = comp; }
    else run_s += expf(comp - run_m);
  }
  return run_m + logf(run_s);
}

// component whose cumulative weight first reaches u (the last one if rounding leaves the total short)
__device__ __forceinline__ int gmm_pick_component(const GmmView& m, size_t row, float u) {
  const float lse = gmm_log_norm(m, row);
  float cum = 0.0f;
  int k = 0;
  for (; k < m.K - 1; ++k) {
    cum += expf(m.logw[row * m.K + k] - lse);
    if (!(cum < u)) break;
  }
  return k;
}

// Draft samples: x[row] = mu_k + sigma_k * noise[row], k = CDF inverse of the weights at u_comp[row].
__global__ void __launch_bounds__(128)
gmm_sample_kernel(int R, int C, GmmView q, const float* __restrict__ u_comp, const float* __restrict__ noise,
                  float* __restrict__ x, int32_t* __restrict__ comp) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= R) return;
  const int k = gmm_pick_component(q, row, u_comp[row]);
  if (lane < C) {
    const size_t o = (static_cast<size_t>(row) * q.K + k) * C + lane;
    x[static_cast<size_t>(row) * C + lane] = fmaf(expf(q.log_sigma[o]), noise[static_cast<size_t>(row) * C + lane], q.mu[o]);
  }
  if (comp && lane == 0) comp[row] = k;
}

// One block per sequence, warp i = draft position i (gamma <= 32): logratio = log p(x) - log q(x), accept iff
// log u <= logratio, n_accept = number of leading accepts.
__global__ void __launch_bounds__(1024)
gmm_verify_kernel(int B, int gamma, int C, GmmView q, GmmView p, const float* __restrict__ x, const float* __restrict__ u,
                  float* __restrict__ logratio, int32_t* __restrict__ n_accept, uint32_t* __restrict__ accept_mask) {
  __shared__ int acc_s[32];
  const int b = blockIdx.x, i = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const size_t row = static_cast<size_t>(b) * gamma + i;
  const float xv = lane < C ? x[row * C + lane] : 0.0f;
  const float lp = gmm_row_logpdf(p, row, C, lane, xv), lq = gmm_row_logpdf(q, row, C, lane, xv);
  const float lr = __fsub_rn(lp, lq);
  if (lane == 0) { logratio[row] = lr; acc_s[i] = logf(u[row]) <= lr ? 1 : 0; }
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t mask = 0u;
    for (int j = 0; j < gamma; ++j) mask |= static_cast<uint32_t>(acc_s[j]) << j;
    const uint32_t rej = ~mask & (gamma >= 32 ? 0xffffffffu : ((1u << gamma) - 1u));
    n_accept[b] = rej ? (__ffs(rej) - 1) : gamma;
    if (accept_mask) accept_mask[b] = mask;
  }
}

// Resampling: one warp per sequence; proposals x' ~ p of the first rejected row, consumed in order,
// alpha_s = max(0, 1 - q(x') / p(x')).
__global__ void __launch_bounds__(128)
gmm_resample_kernel(int B, int gamma, int C, int cap, GmmView q, GmmView p, const int32_t* __restrict__ n_accept,
                    const float* __restrict__ w, const float* __restrict__ xi, const float* __restrict__ v,
                    float* __restrict__ x_new, int32_t* __restrict__ n_prop, uint32_t* __restrict__ flags,
                    int32_t* __restrict__ cap_hits) {
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (b >= B) return;
  const int n = n_accept[b];
  if (n >= gamma) {
    if (lane == 0) { n_prop[b] = 0; flags[b] = 0u; }
    return;
  }
  const size_t row = static_cast<size_t>(b) * gamma + n;
  float xp = 0.0f;
  int k = 0;
  bool done = false;
  for (; k < cap && !done; ++k) {
    const int kc = gmm_pick_component(p, row, w[static_cast<size_t>(b) * cap + k]);
    if (lane < C) {
      const size_t o = (row * p.K + kc) * C + lane;
      xp = fmaf(expf(p.log_sigma[o]), xi[(static_cast<size_t>(b) * cap + k) * C + lane], p.mu[o]);
    }
    const float lp = gmm_row_logpdf(p, row, C, lane, xp), lq = gmm_row_logpdf(q, row, C, lane, xp);
    const float alpha = fmaxf(0.0f, -expm1f(fminf(0.0f, lq - lp)));
    done = v[static_cast<size_t>(b) * cap + k] <= alpha;
  }
  if (lane < C) x_new[static_cast<size_t>(b) * C + lane] = xp;
  if (lane == 0) {
    n_prop[b] = k;
    flags[b] = 1u | (done ? 0u : 2u);
    if (!done) atomicAdd(cap_hits, 1);
  }
}

}  // namespace csd
