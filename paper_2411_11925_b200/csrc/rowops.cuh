// Row-parallel kernels around the GEMM chain: timestep embedding, the per-step boundary kernel
// (eps_hat reduction, classifier-free guidance, DDPM update, input projection, LayerNorm partials,
// condition vector s), and the verification / resampling kernels.
#pragma once
#include "epilogue.cuh"
#include "ptx.cuh"

namespace csd {

// Timestep embedding te[t, :] = Wt2 SiLU(Wt1 tfeat_t + bt1) + bt2 for all T steps: two small fp32 products
// C[m, n] = act(sum_k A[m, k] B[n, k] + bias[n]) in 32 x 32 tiles (each weight row is read once per 32 steps,
// not once per step).
template <bool SILU>
__global__ void __launch_bounds__(256)
small_gemm_nt_kernel(const float* __restrict__ A, const float* __restrict__ B, const float* __restrict__ bias,
                     float* __restrict__ C, int M, int N, int K) {
  __shared__ float As[32][33], Bs[32][33];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;      // 32 x 8 threads, 4 rows of the tile each
  const int m0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
  float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
  for (int k0 = 0; k0 < K; k0 += 32) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = ty * 4 + r, k = k0 + tx;
      As[row][tx] = (m0 + row < M && k < K) ? A[static_cast<size_t>(m0 + row) * K + k] : 0.0f;
      Bs[row][tx] = (n0 + row < N && k < K) ? B[static_cast<size_t>(n0 + row) * K + k] : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 32; ++k) {
      const float b = Bs[tx][k];
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[r] = fmaf(As[ty * 4 + r][k], b, acc[r]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int m = m0 + ty * 4 + r, n = n0 + tx;
    if (m < M && n < N) {
      const float v = acc[r] + bias[n];
      C[static_cast<size_t>(m) * N + n] = SILU ? silu_f(v) : v;
    }
  }
}

template <typename ACT>
__global__ void convert_act_kernel(const float* __restrict__ src, ACT* __restrict__ dst, size_t n) {
  const size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = to_act<ACT>(src[i]);
}

enum StepMode : int { STEP_INIT = 0, STEP_MID = 1, STEP_LAST = 2 };

// Arithmetic of the step boundary, spelled with explicit roundings so that every kernel that
// finishes a step produces the same bits.
// guidance: eps_u + s (eps_c - eps_u)
__device__ __forceinline__ float cfg_combine(float ec, float eu, float scale) { return fmaf(scale, __fsub_rn(ec, eu), eu); }
// Eq. 3 mean: a x - b eps_hat
__device__ __forceinline__ float ddpm_mean(float a, float x, float b, float e) { return fmaf(-b, e, __fmul_rn(a, x)); }
// x_{t-1} = mu + sigma eps
__device__ __forceinline__ float ddpm_sample(float mu, float sigma, float eps) { return fmaf(sigma, eps, mu); }

// h = Win x + bin for the two columns (64 g + lane, 64 g + 32 + lane) of one row, and the (mean, M2)
// LayerNorm partial of the row's 64-column group g (warp-wide; every lane returns the same partial).
// wa / wb: the two columns' rows of Win (16 floats each), ba / bb their biases, xs: the row's x (16).
__device__ __forceinline__ void input_proj_group(const float* wa, const float* wb, float ba, float bb, const float* xs,
                                                 float acc[2], float& mean, float& m2) {
  float a0 = ba, a1 = bb;
#pragma unroll
  for (int c = 0; c < kCPad; ++c) { a0 = fmaf(wa[c], xs[c], a0); a1 = fmaf(wb[c], xs[c], a1); }
  acc[0] = a0; acc[1] = a1;
  float sum = __fadd_rn(a0, a1);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  mean = sum * (1.0f / kStatCols);
  const float d0 = a0 - mean, d1 = a1 - mean;
  m2 = fmaf(d1, d1, __fmul_rn(d0, d0));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m2 += __shfl_xor_sync(0xffffffffu, m2, o);
}

struct StepParams {
  int R, cfg, C, W, NT;          // token rows, guidance flag, token dim, width, number of column tiles
  float cfg_scale, a, b, sigma;  // coefficients of the step being finished (t)
  int sample_last;               // STEP_LAST: also draw x0 = mu1 + sigma eps
  const float* epart;            // [Rh, NT, 16] eps_hat partial sums of step t
  const float* bout;             // [16] (zero padded)
  const float* eps_t;            // [R, C] noise of step t
  const float* x_src;            // STEP_INIT: x_T
  float* x;                      // [R, C] current state (in/out)
  float *x0, *mu1, *x1;          // STEP_LAST outputs (x0, x1 may be null)
  const float* win;              // [W, 16] (zero padded), bin [W]
  const float* bin;
  const float* cz;               // [Rh, W]
  const float* te_next;          // [W] embedding of the step being prepared
  float* h;                      // [Rh, W]
  float* stats;                  // [Rh, W/64, 2]
  void* s;                       // [Rh, W] activations: s of the step te_next belongs to (null: none)
  void* s_b;                     // a second s to prepare (first boundary only), with its embedding te_b
  const float* te_b;
  float* traj_x;                 // TRAJ kernels: where the state this boundary produces is recorded ([R, C])
  float* traj_mu;                // TRAJ kernels: where the mean of the step being finished is recorded ([R, C])
  int* status;                   // set to 1 when a mean or state of this step is not finite (csd_sync reports it)
  // learned-variance heads (LV kernels): epart rows are 32 wide, [eps partials | variance-parameter partials]
  float lv_min, lv_max;          // bounds of the log-variance at the step being finished
  float* lv1;                    // STEP_LAST: [R, C] log-variance of the last step
  float* half_logdet;            // [R]: (1/2) sum over steps t >= 2 and coordinates of the log-variance (zeroed by STEP_INIT)
};

// log-variance of one coordinate from the head's variance output w: lv_min + (w + 1)/2 (lv_max - lv_min)
__device__ __forceinline__ float lv_interp(float w, float lv_min, float lv_max) {
  return fmaf(__fmul_rn(0.5f, __fadd_rn(w, 1.0f)), __fsub_rn(lv_max, lv_min), lv_min);
}

// RB token rows per block.  Finishes step t (unless STEP_INIT) and prepares the next one:
//   eps_hat = sum of tile partials + bout; guidance; mu = a x - b eps_hat; x <- mu + sigma eps_t
//   h = Win x + bin (same for both guidance rows), LayerNorm partials per 64 columns,
//   s = SiLU(cz + te_next) of the step after that (s is double-buffered, see the host code).
// With one row per block the kernel is bound by re-reading Win (64 B per column and row) through L1; RB = 4 reads a
// group's columns once for four rows.  The arithmetic of a row does not depend on RB.
// TRAJ: also record the whole trajectory (every state and every mean), for the single-path ratio of Eq. 2.
// LV: the head also predicts its transition's diagonal variance (Eq. 3 in its general form): the noise is scaled per
// coordinate by exp(lv / 2), the row's half log-determinant is accumulated for Sigma of Eq. 7.
template <typename ACT, int RB, bool TRAJ = false, bool LV = false>
__global__ void __launch_bounds__(256, RB == 4 ? 3 : 0) step_kernel(StepParams p, int mode) {
  constexpr int EPW = LV ? kCPad2 : kCPad;
  __shared__ float xs[RB][kCPad];
  __shared__ float eh[RB][2][kCPad];
  __shared__ float wv[LV ? RB : 1][kCPad];
  const int r0 = blockIdx.x * RB, tid = threadIdx.x;
  const int nrep = p.cfg ? 2 : 1;
  const int nrow = min(RB, p.R - r0);
  griddep_wait();
  if (tid == 0) griddep_launch_dependents();
  if (mode == STEP_INIT) {
    if (tid < RB * kCPad) {
      const int rr = tid / kCPad, c = tid % kCPad;
      float v = 0.0f;
      if (rr < nrow && c < p.C) {
        v = p.x_src[static_cast<size_t>(r0 + rr) * p.C + c];
        p.x[static_cast<size_t>(r0 + rr) * p.C + c] = v;
        if (TRAJ) p.traj_x[static_cast<size_t>(r0 + rr) * p.C + c] = v;
        if (LV && c == 0) p.half_logdet[r0 + rr] = 0.0f;
      }
      xs[rr][c] = v;
    }
    __syncthreads();
  } else {
    if (tid < RB * 2 * kCPad) {
      const int c = tid % kCPad, rep = (tid / kCPad) & 1, rr = tid / (2 * kCPad);
      if (rr < nrow && rep < nrep) {
        const float* e = p.epart + (static_cast<size_t>(r0 + rr + rep * p.R) * p.NT) * EPW + c;
        float acc = 0.0f;
        for (int nt = 0; nt < p.NT; ++nt) acc += e[nt * EPW];
        eh[rr][rep][c] = acc + p.bout[c];
        if (LV && rep == 0) {       // the variance parameter is the conditional row's own
          float accv = 0.0f;
          for (int nt = 0; nt < p.NT; ++nt) accv += e[nt * EPW + kCPad];
          wv[rr][c] = accv + p.bout[kCPad + c];
        }
      }
    }
    __syncthreads();
    if (tid < RB * kCPad) {
      const int rr = tid / kCPad, c = tid % kCPad;
      float xn = 0.0f;
      if (rr < nrow && c < p.C) {
        const size_t o = static_cast<size_t>(r0 + rr) * p.C + c;
        float e = eh[rr][0][c];
        if (p.cfg) e = cfg_combine(eh[rr][0][c], eh[rr][1][c], p.cfg_scale);
        const float xo = p.x[o];
        const float mu = ddpm_mean(p.a, xo, p.b, e);
        float sigma = p.sigma, lv = 0.0f;
        if (LV) { lv = lv_interp(wv[rr][c], p.lv_min, p.lv_max); sigma = expf(0.5f * lv); }
        xn = ddpm_sample(mu, sigma, p.eps_t[o]);
        // an activation beyond the 16-bit operand range became inf further up and arrives here as inf or NaN
        if (!(fabsf(xn) <= 3.0e38f)) *p.status = 1;
        if (LV && mode == STEP_LAST) p.lv1[o] = lv;
        if (mode == STEP_LAST) {
          p.mu1[o] = mu;
          if (p.x1) p.x1[o] = xo;
          if (p.sample_last && p.x0) p.x0[o] = xn;
        } else {
          p.x[o] = xn;
          if (TRAJ) { p.traj_x[o] = xn; p.traj_mu[o] = mu; }
        }
      }
      xs[rr][c] = xn;
      if (LV && mode != STEP_LAST) {
        // (1/2) sum_d lv of this step, coordinates in order (lanes 0..15 of a half-warp hold one row)
        float hsum = (rr < nrow && c < p.C) ? 0.5f * lv_interp(wv[rr][c], p.lv_min, p.lv_max) : 0.0f;
        constexpr unsigned kRowLanes = RB * kCPad >= 32 ? 0xffffffffu : 0x0000ffffu;   // threads inside this branch
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) hsum += __shfl_xor_sync(kRowLanes, hsum, o);
        if (rr < nrow && c == 0) p.half_logdet[r0 + rr] += hsum;
      }
    }
    if (mode == STEP_LAST) return;
    __syncthreads();
  }
  // prepare: each warp handles 64 consecutive columns at a time (lane, lane + 32): one LayerNorm partial
  const int lane = tid & 31, warp = tid >> 5, nwarp = blockDim.x >> 5;
  ACT* s = reinterpret_cast<ACT*>(p.s);
  ACT* s_b = reinterpret_cast<ACT*>(p.s_b);
  for (int g = warp; g < p.W / kStatCols; g += nwarp) {
    float wa[kCPad], wb[kCPad];
    const int na = g * kStatCols + lane, nb = na + 32;
#pragma unroll
    for (int c4 = 0; c4 < kCPad / 4; ++c4) {
      const float4 qa = reinterpret_cast<const float4*>(p.win + static_cast<size_t>(na) * kCPad)[c4];
      const float4 qb = reinterpret_cast<const float4*>(p.win + static_cast<size_t>(nb) * kCPad)[c4];
      wa[4 * c4] = qa.x; wa[4 * c4 + 1] = qa.y; wa[4 * c4 + 2] = qa.z; wa[4 * c4 + 3] = qa.w;
      wb[4 * c4] = qb.x; wb[4 * c4 + 1] = qb.y; wb[4 * c4 + 2] = qb.z; wb[4 * c4 + 3] = qb.w;
    }
    const float ba = p.bin[na], bb = p.bin[nb];
    float te[2] = {0.0f, 0.0f}, teb[2] = {0.0f, 0.0f};
    if (s) { te[0] = p.te_next[na]; te[1] = p.te_next[nb]; }
    if (s_b) { teb[0] = p.te_b[na]; teb[1] = p.te_b[nb]; }
    // every cz value of the group first: the loads are independent, but behind the stores below the compiler must
    // assume they are not, and each row would wait for its own trip to memory
    float czv[RB][2][2];
#pragma unroll
    for (int rr = 0; rr < RB; ++rr)
#pragma unroll
      for (int rep = 0; rep < 2; ++rep)
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const size_t row = static_cast<size_t>(r0 + rr) + static_cast<size_t>(rep) * p.R;
          czv[rr][rep][j] = (rr < nrow && rep < nrep && (s || s_b)) ? __ldg(p.cz + row * p.W + g * kStatCols + j * 32 + lane) : 0.0f;
        }
#pragma unroll
    for (int rr = 0; rr < RB; ++rr) {
      if (rr >= nrow) break;
      float acc[2], mean, m2;
      input_proj_group(wa, wb, ba, bb, xs[rr], acc, mean, m2);
#pragma unroll
      for (int rep = 0; rep < 2; ++rep) {
        if (rep >= nrep) break;
        const size_t row = static_cast<size_t>(r0 + rr) + static_cast<size_t>(rep) * p.R;
        if (lane == 0)
          reinterpret_cast<float2*>(p.stats)[row * (p.W / kStatCols) + g] = make_float2(mean, m2);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int n = g * kStatCols + j * 32 + lane;
          p.h[row * p.W + n] = acc[j];
          if (s) s[row * p.W + n] = to_act<ACT>(silu_f(czv[rr][rep][j] + te[j]));
          if (s_b) s_b[row * p.W + n] = to_act<ACT>(silu_f(czv[rr][rep][j] + teb[j]));
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Single-path ratio (Eq. 2): the target head scores the DRAFT's trajectory, so its T evaluations do not depend
// on one another and several steps are evaluated as one batch of rows.  Token row r' = j * Rin + r of a pass is
// row r of trajectory slot j0 + j (timestep t = T - j0 - j); with guidance its head rows are r' and Rtok + r'.
struct BatchParams {
  int Rin, Rtok, cfg, C, W, NT, T, j0;   // rows per step, token rows of the pass, ..., first trajectory slot
  float cfg_scale;
  const float* sched;    // device [5, T] of the target / draft pair: a, b, log-constant, 1/(2 sigma_p^2), 1/(2 sigma_q^2)
  const float* traj_x;   // [T + 1, Rin, C]: slot j holds x_{T-j}
  const float* win;      // [W, 16] (zero padded), bin [W]
  const float* bin;
  const float* cz;       // [Rin (1 + cfg), W]: one condition projection per row, shared by all steps
  const float* te;       // [T, W]
  float* h;              // [Rh, W]
  float* stats;          // [Rh, W/64, 2]
  void* s;               // [Rh, W] activations
  const float* epart;    // [Rh, NT, 16] eps_hat partial sums
  const float* bout;     // [16]
  float* mu_p;           // [Rtok, C] out: mean of the target's transition at the draft's state
  int* status;           // set to 1 when a mean is not finite
};

// Prepares a pass: h = Win x + bin, its LayerNorm partials and s = SiLU(cz + te_t), four token rows per block,
// with the arithmetic of step_kernel (the same device functions), so a row gets the bits it gets there.
template <typename ACT>
__global__ void __launch_bounds__(256) batch_prepare_kernel(BatchParams p) {
  constexpr int RB = 4;
  __shared__ float xs[RB][kCPad];
  const int r0 = blockIdx.x * RB, tid = threadIdx.x;
  const int nrep = p.cfg ? 2 : 1;
  const int nrow = min(RB, p.Rtok - r0);
  griddep_wait();
  if (tid == 0) griddep_launch_dependents();
  if (tid < RB * kCPad) {
    const int rr = tid / kCPad, c = tid % kCPad;
    float v = 0.0f;
    if (rr < nrow && c < p.C) v = p.traj_x[(static_cast<size_t>(p.j0) * p.Rin + r0 + rr) * p.C + c];
    xs[rr][c] = v;
  }
  __syncthreads();
  const int lane = tid & 31, warp = tid >> 5, nwarp = blockDim.x >> 5;
  ACT* s = reinterpret_cast<ACT*>(p.s);
  for (int g = warp; g < p.W / kStatCols; g += nwarp) {
    float wa[kCPad], wb[kCPad];
    const int na = g * kStatCols + lane, nb = na + 32;
#pragma unroll
    for (int c4 = 0; c4 < kCPad / 4; ++c4) {
      const float4 qa = reinterpret_cast<const float4*>(p.win + static_cast<size_t>(na) * kCPad)[c4];
      const float4 qb = reinterpret_cast<const float4*>(p.win + static_cast<size_t>(nb) * kCPad)[c4];
      wa[4 * c4] = qa.x; wa[4 * c4 + 1] = qa.y; wa[4 * c4 + 2] = qa.z; wa[4 * c4 + 3] = qa.w;
      wb[4 * c4] = qb.x; wb[4 * c4 + 1] = qb.y; wb[4 * c4 + 2] = qb.z; wb[4 * c4 + 3] = qb.w;
    }
    const float ba = p.bin[na], bb = p.bin[nb];
    // every cz and te value of the group first: independent loads in flight together (one trip to memory per
    // group instead of one per row)
    float czv[RB][2][2], tev[RB][2];
#pragma unroll
    for (int rr = 0; rr < RB; ++rr) {
      const int rt = min(r0 + rr, p.Rtok - 1), j = rt / p.Rin, ri = rt - j * p.Rin;
      const float* te = p.te + static_cast<size_t>(p.T - 1 - p.j0 - j) * p.W;
      tev[rr][0] = te[na]; tev[rr][1] = te[nb];
#pragma unroll
      for (int rep = 0; rep < 2; ++rep) {
        const size_t zrow = static_cast<size_t>(ri) + static_cast<size_t>(rep < nrep ? rep : 0) * p.Rin;
        czv[rr][rep][0] = __ldg(p.cz + zrow * p.W + na);
        czv[rr][rep][1] = __ldg(p.cz + zrow * p.W + nb);
      }
    }
#pragma unroll
    for (int rr = 0; rr < RB; ++rr) {
      if (rr >= nrow) break;
      const int rt = r0 + rr;
      float acc[2], mean, m2;
      input_proj_group(wa, wb, ba, bb, xs[rr], acc, mean, m2);
#pragma unroll
      for (int rep = 0; rep < 2; ++rep) {
        if (rep >= nrep) break;
        const size_t row = static_cast<size_t>(rt) + static_cast<size_t>(rep) * p.Rtok;
        if (lane == 0)
          reinterpret_cast<float2*>(p.stats)[row * (p.W / kStatCols) + g] = make_float2(mean, m2);
        p.h[row * p.W + na] = acc[0];
        p.h[row * p.W + nb] = acc[1];
        s[row * p.W + na] = to_act<ACT>(silu_f(czv[rr][rep][0] + tev[rr][0]));
        s[row * p.W + nb] = to_act<ACT>(silu_f(czv[rr][rep][1] + tev[rr][1]));
      }
    }
  }
}

// Finishes a pass: eps_hat = sum of tile partials + bout, guidance, mu^p_t = a_t x_t - b_t eps_hat (Eq. 3 mean),
// 16 token rows per block of 256 threads (thread = row, coordinate).
__global__ void __launch_bounds__(256) batch_finish_kernel(BatchParams p) {
  const int rt = blockIdx.x * 16 + (threadIdx.x >> 4), c = threadIdx.x & 15;
  griddep_wait();
  if (rt >= p.Rtok || c >= p.C) return;
  float e[2] = {0.0f, 0.0f};
  for (int rep = 0; rep < (p.cfg ? 2 : 1); ++rep) {
    const float* ep = p.epart + (static_cast<size_t>(rt) + static_cast<size_t>(rep) * p.Rtok) * p.NT * kCPad + c;
    float acc = 0.0f;
    for (int nt = 0; nt < p.NT; ++nt) acc += ep[nt * kCPad];
    e[rep] = acc + p.bout[c];
  }
  const float eh = p.cfg ? cfg_combine(e[0], e[1], p.cfg_scale) : e[0];
  const int ti = p.T - 1 - p.j0 - rt / p.Rin;   // t - 1
  const float x = p.traj_x[(static_cast<size_t>(p.j0) * p.Rin + rt) * p.C + c];
  const float mu = ddpm_mean(p.sched[ti], x, p.sched[p.T + ti], eh);
  if (!(fabsf(mu) <= 3.0e38f)) *p.status = 1;
  p.mu_p[static_cast<size_t>(rt) * p.C + c] = mu;
}

// Per-step terms of the log-ratio of Eq. 2 for the steps of one pass, one thread per (step, token row):
//   term_t = C (log sigma_q,t - log sigma_p,t) - |x_{t-1} - mu^p_t|^2 / (2 sigma_p,t^2) + |x_{t-1} - mu^q_t|^2 / (2 sigma_q,t^2).
// The two quadratic forms are rounded separately, so identical means give a term of exactly zero.
__global__ void __launch_bounds__(128)
single_path_terms_kernel(int Rin, int C, int T, int j0, int nsteps, const float* __restrict__ sched,
                         const float* __restrict__ traj_x, const float* __restrict__ traj_mu,
                         const float* __restrict__ mu_p, float* __restrict__ terms) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= nsteps * Rin) return;
  const int j = i / Rin, r = i - j * Rin;
  const int ti = T - 1 - j0 - j;
  const float* xn = traj_x + (static_cast<size_t>(j0 + j + 1) * Rin + r) * C;
  const float* mq = traj_mu + (static_cast<size_t>(j0 + j) * Rin + r) * C;
  const float* mp = mu_p + static_cast<size_t>(i) * C;
  float dp = 0.0f, dq = 0.0f;
  for (int c = 0; c < C; ++c) {
    const float x = xn[c];
    const float ep = x - mp[c], eq = x - mq[c];
    dp = fmaf(ep, ep, dp);
    dq = fmaf(eq, eq, dq);
  }
  terms[static_cast<size_t>(j0 + j) * Rin + r] =
      sched[2 * T + ti] + __fsub_rn(__fmul_rn(dq, sched[4 * T + ti]), __fmul_rn(dp, sched[3 * T + ti]));
}

// Sum of the T terms in trajectory order (in double, so the order of magnitude of the early terms does not cost the
// late ones their digits), then the accept test and prefix scan of Alg. 1: one warp per sequence.
__global__ void __launch_bounds__(128)
single_path_accept_kernel(int B, int gamma, int T, const float* __restrict__ terms, const float* __restrict__ u,
                          float* __restrict__ logratio, int32_t* __restrict__ n_accept,
                          uint32_t* __restrict__ accept_mask) {
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (b >= B) return;
  bool ok = true;
  if (lane < gamma) {
    const size_t row = static_cast<size_t>(b) * gamma + lane;
    const size_t R = static_cast<size_t>(B) * gamma;
    double total = 0.0;
    for (int j = 0; j < T; ++j) total += static_cast<double>(terms[j * R + row]);
    const float lr = static_cast<float>(total);
    logratio[row] = lr;
    ok = logf(u[row]) <= lr;
  }
  const uint32_t ballot = __ballot_sync(0xffffffffu, ok);
  if (lane == 0) {
    const uint32_t rej = ~ballot;
    int n = rej ? (__ffs(rej) - 1) : gamma;
    if (n > gamma) n = gamma;
    n_accept[b] = n;
    if (accept_mask) accept_mask[b] = (gamma >= 32) ? ballot : (ballot & ((1u << gamma) - 1u));
  }
}

// ---------------------------------------------------------------------------------------------
// Verification: one warp per sequence, lane i = draft position i (gamma <= 32).
//   logratio = log_sigma + C (log sq1 - log sp1) - |x0 - mu_p|^2 / (2 sp1^2) + |x0 - mu_q|^2 / (2 sq1^2)
//   accept iff log u <= logratio;  n_accept = number of leading accepts (ballot + find-first-set).
__global__ void __launch_bounds__(128)
accept_scan_kernel(int B, int gamma, int C, float log_const, float inv2vp, float inv2vq,
                   const float* __restrict__ x0, const float* __restrict__ mu_q,
                   const float* __restrict__ mu_p, const float* __restrict__ u,
                   float* __restrict__ logratio, int32_t* __restrict__ n_accept,
                   uint32_t* __restrict__ accept_mask, const float* __restrict__ offset = nullptr) {
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (b >= B) return;
  bool acc = true;  // lanes beyond gamma do not reject
  if (lane < gamma) {
    const size_t row = static_cast<size_t>(b) * gamma + lane;
    float dp = 0.0f, dq = 0.0f;
    for (int c = 0; c < C; ++c) {
      const float x = x0[row * C + c];
      const float ep = x - mu_p[row * C + c];
      const float eq = x - mu_q[row * C + c];
      dp = fmaf(ep, ep, dp);
      dq = fmaf(eq, eq, dq);
    }
    // Both products are rounded separately (no FMA contraction), so that identical draft and target
    // means give a difference of exactly zero.
    float lr = log_const + __fsub_rn(__fmul_rn(dq, inv2vq), __fmul_rn(dp, inv2vp));
    if (offset) lr = __fadd_rn(lr, offset[row]);   // terms of the steps t >= 2 when the noise is not shared
    logratio[row] = lr;
    acc = logf(u[row]) <= lr;
  }
  const uint32_t ballot = __ballot_sync(0xffffffffu, acc);
  if (lane == 0) {
    const uint32_t rej = ~ballot;
    int n = rej ? (__ffs(rej) - 1) : gamma;
    if (n > gamma) n = gamma;
    n_accept[b] = n;
    if (accept_mask) accept_mask[b] = (gamma >= 32) ? ballot : (ballot & ((1u << gamma) - 1u));
  }
}

// Without trajectory alignment the exponentials of the steps t >= 2 of Eq. 4 do not cancel: x^m_{t-1} - mu^m_t =
// sigma_m,t eps^m_t, so step t contributes (|eps^q_t|^2 - |eps^p_t|^2) / 2 beyond the Sigma term.  One thread per
// token row, steps in order, double accumulation; identical noise gives exactly 0.
__global__ void __launch_bounds__(128)
noise_norm_term_kernel(int R, int C, int T, const float* __restrict__ eps_q, const float* __restrict__ eps_p,
                       float* __restrict__ offset) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= R) return;
  double total = 0.0;
  for (int t = 1; t < T; ++t) {   // slices 1..T-1 = steps 2..T
    const float* a = eps_q + (static_cast<size_t>(t) * R + r) * C;
    const float* b = eps_p + (static_cast<size_t>(t) * R + r) * C;
    float nq = 0.0f, np = 0.0f;
    for (int c = 0; c < C; ++c) { nq = fmaf(a[c], a[c], nq); np = fmaf(b[c], b[c], np); }
    total += 0.5 * (static_cast<double>(nq) - static_cast<double>(np));
  }
  offset[r] = static_cast<float>(total);
}

// All-accepted branch of Alg. 1: sequence b keeps its sample of position gamma + 1 only if n_accept[b] == gamma.
__global__ void __launch_bounds__(256)
bonus_select_kernel(int B, int C, int gamma, const int32_t* __restrict__ n_accept, const float* __restrict__ x0,
                    float* __restrict__ x_bonus, uint32_t* __restrict__ taken) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * C) return;
  const int b = i / C;
  const bool all = n_accept[b] >= gamma;
  if (all) x_bonus[i] = x0[i];
  if (taken && i == b * C) taken[b] = all ? 1u : 0u;
}

// Verification with predicted diagonal variances.  Per token  log Sigma = half_logdet_q - half_logdet_p  (Eq. 7: the
// product over t >= 2 of sqrt|Sigma_q,t| / sqrt|Sigma_p,t|, accumulated by the two chains), and
//   logratio = log Sigma + log N(x0; mu_p, diag(exp(lv_p))) - log N(x0; mu_q, diag(exp(lv_q)))      (Eq. 8).
// Each model's exponent-plus-normaliser sum is formed by the same instruction sequence, so identical draft and target
// values give a difference of exactly zero.
__device__ __forceinline__ float diag_neg_logpdf(const float* x, const float* mu, const float* lv, int C) {
  float acc = 0.0f;     // sum_d [ lv_d / 2 + (x - mu)_d^2 / (2 exp(lv_d)) ]
  for (int c = 0; c < C; ++c) {
    const float e = x[c] - mu[c];
    acc = __fadd_rn(acc, __fadd_rn(__fmul_rn(0.5f, lv[c]), __fmul_rn(__fmul_rn(0.5f, __fmul_rn(e, e)), expf(-lv[c]))));
  }
  return acc;
}

__global__ void __launch_bounds__(128)
accept_scan_lv_kernel(int B, int gamma, int C, const float* __restrict__ x0, const float* __restrict__ mu_q,
                      const float* __restrict__ lv_q, const float* __restrict__ hld_q, const float* __restrict__ mu_p,
                      const float* __restrict__ lv_p, const float* __restrict__ hld_p, const float* __restrict__ u,
                      float* __restrict__ logratio, float* __restrict__ log_sigma_rows, int32_t* __restrict__ n_accept,
                      uint32_t* __restrict__ accept_mask) {
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (b >= B) return;
  bool acc = true;
  if (lane < gamma) {
    const size_t row = static_cast<size_t>(b) * gamma + lane;
    const float ls = __fsub_rn(hld_q[row], hld_p[row]);
    const float nq = diag_neg_logpdf(x0 + row * C, mu_q + row * C, lv_q + row * C, C);
    const float np = diag_neg_logpdf(x0 + row * C, mu_p + row * C, lv_p + row * C, C);
    const float lr = __fadd_rn(ls, __fsub_rn(nq, np));
    log_sigma_rows[row] = ls;
    logratio[row] = lr;
    acc = logf(u[row]) <= lr;
  }
  const uint32_t ballot = __ballot_sync(0xffffffffu, acc);
  if (lane == 0) {
    const uint32_t rej = ~ballot;
    int n = rej ? (__ffs(rej) - 1) : gamma;
    if (n > gamma) n = gamma;
    n_accept[b] = n;
    if (accept_mask) accept_mask[b] = (gamma >= 32) ? ballot : (ballot & ((1u << gamma) - 1u));
  }
}

// Corollary 1 with diagonal final-step covariances: x' = mu_p + exp(lv_p / 2) xi, alpha_s = max(0, 1 - q(x') / (Sigma p(x')))
// with the rejected token's own Sigma; one warp per sequence, lane c < C = coordinate.
__global__ void __launch_bounds__(128)
resample_lv_kernel(int B, int gamma, int C, int cap, const float* __restrict__ log_sigma_rows,
                   const int32_t* __restrict__ n_accept, const float* __restrict__ mu_p, const float* __restrict__ lv_p,
                   const float* __restrict__ mu_q, const float* __restrict__ lv_q, const float* __restrict__ xi,
                   const float* __restrict__ v, float* __restrict__ x_new, int32_t* __restrict__ n_prop,
                   uint32_t* __restrict__ flags, int32_t* __restrict__ cap_hits) {
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (b >= B) return;
  const int n = n_accept[b];
  if (n >= gamma) {
    if (lane == 0) { n_prop[b] = 0; flags[b] = 0u; }
    return;
  }
  const size_t row = static_cast<size_t>(b) * gamma + n;
  const bool on = lane < C;
  const float mp = on ? mu_p[row * C + lane] : 0.0f, mq = on ? mu_q[row * C + lane] : 0.0f;
  const float lp_d = on ? lv_p[row * C + lane] : 0.0f, lq_d = on ? lv_q[row * C + lane] : 0.0f;
  const float sp = expf(0.5f * lp_d), ivp = 0.5f * expf(-lp_d), ivq = 0.5f * expf(-lq_d);
  const float ls = log_sigma_rows[row];
  float hl = on ? 0.5f * (lq_d - lp_d) : 0.0f;      // (1/2) sum_d (lv_q - lv_p): the normalisers' part of lq - lp ... negated below
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) hl += __shfl_xor_sync(0xffffffffu, hl, o);
  float xp = 0.0f;
  int k = 0;
  bool done = false;
  for (; k < cap && !done; ++k) {
    const float z = on ? xi[(static_cast<size_t>(b) * cap + k) * C + lane] : 0.0f;
    xp = mp + sp * z;
    float ep = on ? (xp - mp) : 0.0f, eq = on ? (xp - mq) : 0.0f;
    ep = ep * ep * ivp; eq = eq * eq * ivq;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      ep += __shfl_xor_sync(0xffffffffu, ep, o);
      eq += __shfl_xor_sync(0xffffffffu, eq, o);
    }
    // lq - lp = -(1/2) sum lv_q - eq + (1/2) sum lv_p + ep = -hl - eq + ep
    const float alpha = fmaxf(0.0f, -expm1f(fminf(0.0f, (ep - eq) - hl - ls)));
    done = v[static_cast<size_t>(b) * cap + k] <= alpha;
  }
  if (on) x_new[static_cast<size_t>(b) * C + lane] = xp;
  if (lane == 0) {
    n_prop[b] = k;
    flags[b] = 1u | (done ? 0u : 2u);
    if (!done) atomicAdd(cap_hits, 1);
  }
}

// Self-test of the bounded waits: one thread waits on a barrier on which nobody ever arrives, so the wait runs
// into the limit (csd_set_wait_limit), gives up and records role 4, site 1 in the context's error word.  Nothing
// else happens: no fault, no trap, no wait beyond the limit.
__global__ void wait_timeout_selftest_kernel(int* err) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) { mbar_init(&bar, 1); fence_mbar_init(); }
  __syncthreads();
  if (threadIdx.x == 0 && !ch_wait<false>(&bar, 0, err)) ch_fail(err, 4, 1, 0);
}

// Resampling: one warp per sequence, lane c < C = coordinate.  Proposals are consumed in order.
__global__ void __launch_bounds__(128)
resample_kernel(int B, int gamma, int C, int cap, float log_sigma, float sp1, float sq1,
                float log_sp1, float log_sq1, const int32_t* __restrict__ n_accept,
                const float* __restrict__ mu_p, const float* __restrict__ mu_q,
                const float* __restrict__ xi, const float* __restrict__ v,
                float* __restrict__ x_new, int32_t* __restrict__ n_prop,
                uint32_t* __restrict__ flags, int32_t* __restrict__ cap_hits) {
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (b >= B) return;
  const int n = n_accept[b];
  if (n >= gamma) {
    if (lane == 0) { n_prop[b] = 0; flags[b] = 0u; }
    return;
  }
  const size_t row = static_cast<size_t>(b) * gamma + n;
  const float mp = (lane < C) ? mu_p[row * C + lane] : 0.0f;
  const float mq = (lane < C) ? mu_q[row * C + lane] : 0.0f;
  const float inv2vp = 0.5f / (sp1 * sp1), inv2vq = 0.5f / (sq1 * sq1);
  float xp = 0.0f;
  int k = 0;
  bool done = false;
  for (; k < cap && !done; ++k) {
    const float z = (lane < C) ? xi[(static_cast<size_t>(b) * cap + k) * C + lane] : 0.0f;
    xp = mp + sp1 * z;
    float ep = (lane < C) ? (xp - mp) : 0.0f;
    float eq = (lane < C) ? (xp - mq) : 0.0f;
    ep *= ep; eq *= eq;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      ep += __shfl_xor_sync(0xffffffffu, ep, o);
      eq += __shfl_xor_sync(0xffffffffu, eq, o);
    }
    const float lp = -C * log_sp1 - ep * inv2vp;
    const float lq = -C * log_sq1 - eq * inv2vq;
    const float alpha = fmaxf(0.0f, -expm1f(fminf(0.0f, lq - log_sigma - lp)));
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
