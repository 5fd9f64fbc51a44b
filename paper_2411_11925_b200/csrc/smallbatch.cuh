// One persistent kernel for a whole denoising chain (all T steps of Eq. 3 for one head) when the call has few rows:
// the regime Alg. 1 forces on the draft model, whose tokens x_i ~ q_i come one position at a time.  With at most
// 128 head rows a layer is a single row tile; the layer-by-layer kernels then keep 8-16 SMs busy and pay a kernel
// boundary per layer.  Here the whole GPU streams each layer's weights and nothing ever waits for the whole grid:
//
//   * A head is a per-token MLP: token rows never exchange data.  The rows are cut into groups of 16 (with guidance:
//     8 tokens, the conditional rows and their unconditional twins), and a thread-block cluster of 8 CTAs owns one
//     group for all layers and all steps.  The only synchronisation on the dependent path is that cluster's own
//     hardware barrier, once per layer.
//   * Operands are swapped: the weights are the M operand of the MMA (CTA n of a cluster owns output columns
//     [128 n, 128 n + 128) of every layer), the group's 16 rows its N.  A CTA streams its [128 x W] weight slab
//     through a TMA ring of two 64 KB stages that runs ahead across layers (weights depend on nothing), so after the
//     barrier only the group's 16 x W activations (32 KB at W = 1024) have to arrive before the MMAs start; a stage
//     holds four k-blocks, because the issuing thread pays a few hundred cycles per barrier round trip.
//   * Every product of the condition vector s_t (AdaLN gate and scale, the LayerNorm-folded first-layer terms P1 | P2
//     of fold.cuh, the final shift | scale) does not depend on x_t: the remaining clusters ("early" CTAs) compute
//     them a step ahead as full tiles (all 128 rows, full K) and leave them in a two-slot buffer in global memory.
//   * Per step a group runs 2 L product phases and a boundary in two halves: token-parallel, finish the step (final
//     modulate, output projection, guidance, Eq. 3 update); column-parallel, prepare the next (input projection,
//     LayerNorm partials, a' of block 0).
//
// All blocks run in the folded form of fold.cuh (v = SiLU(rstd (a' W1^T - mean (P1 + c1)) + P2 + c2) with
// a' = h (1 + scale)), block 0 included, so results agree with the layer kernels within the trajectory tolerance,
// not bit for bit.  Rows are kept in the kernel's own order (group after group).  Every software wait is bounded; once
// one gives up it raises the context's status word, every later wait returns at once and the kernel winds down
// through its remaining barriers without doing work.
#pragma once
#include "fold.cuh"

namespace csd {

constexpr int kSbCluster = 8;
constexpr int kSbThreads = 192;          // warp 0: TMA, warp 1: MMA, warps 2..5: workers
constexpr int kSbWorkers = 128;
constexpr int kSbRows = 128;             // rows per call (padded): 8 groups of 16
constexpr int kSbGroup = 16;             // rows per group = MMA N of the dependent products
constexpr int kSbMaxW = 1536;            // at most two column tiles per CTA
constexpr int kSbKps = 4;                // k-blocks (16 KB weight tiles) per ring stage: one barrier round trip per 64 KB
constexpr int kSbStages = 2;             // dependent CTAs: ring stages
constexpr int kSbActBytes = kSbGroup * kSbMaxW * 2;            // the group's activations, [k-block][16 rows][64]
constexpr int kSbEarlyStages = 6;        // early CTAs: ring of [A 16 KB | B 16 KB]
constexpr int kSbStageBytes = kSbKps * 16384;
constexpr int kSbDepBytes = kSbStages * kSbStageBytes + kSbActBytes;
constexpr int kSbEarlyBytes = kSbEarlyStages * 32768;
constexpr int kSbSmemBytes = 1024 + (kSbDepBytes > kSbEarlyBytes ? kSbDepBytes : kSbEarlyBytes) + 4096;
static_assert(kSbSmemBytes <= 227 * 1024, "shared memory of the small-batch kernel");

struct SbTask { int map, row, col, pad; };   // early-product tile: tensor map index, first weight row, first mods column

struct SbParams {
  int R, Rh, cfg, W, L, T, C, sample_last;
  float cfg_scale;
  int nd, ne;                   // clusters: row groups of the dependent chain, early products
  int ntasks, nm;               // early tiles per step; mods columns per row = (5 L + 2) W
  const CUtensorMap* maps;      // device: W1_0, W2_0, .., W1_{L-1}, W2_{L-1} (boxes 64 x 128), then the early matrices
  const SbTask* tasks;          // device [ntasks]
  const float* sched;           // device [3 T]: a, b, sigma
  const float* const* bias;     // device: per block c1, c2, gate bias, b2, scale bias; then final shift bias, scale bias
  float* mods;                  // [2][128][nm] fp32: products of s_t of the step with parity t & 1 (kernel row order)
  float* h;                     // [128, W]       (kernel row order, as are stats, ap, v)
  float* stats;                 // [128, W/64, 2]
  void* ap;                     // [128, W] a' = h (1 + scale), operand format
  void* v;                      // [128, W]
  float* x;                     // [R, C]
  const float *win, *bin, *wout_t, *bout;
  const float *x_T, *eps;
  float *x0, *mu1, *x1;
  int* sync;                    // [0] steps finished, summed over the row groups; [1 + t] early tiles finished for step t
  int* err;
  int* status;
};

// Kernel row order: group g holds rows 16 g .. 16 g + 15.  Without guidance row rho is token rho; with guidance group g
// holds tokens 8 g .. 8 g + 7, conditional rows first, then their unconditional twins.
__host__ __device__ __forceinline__ int sb_row_token(int rho, int cfg, int* rep) {
  if (!cfg) { *rep = 0; return rho; }
  *rep = (rho >> 3) & 1;
  return (rho >> 4) * 8 + (rho & 7);
}

__device__ __forceinline__ int sb_ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// One thread waits until *p >= target (bounded; also gives up once the context's status word is up).
__device__ __forceinline__ bool sb_wait_count(const int* p, int target, const int* err) {
  long long t0 = 0;
  uint32_t spins = 0;
  for (;;) {
    if (sb_ld_acquire(p) >= target) return true;
    if ((++spins & 255u) == 0u) {
      if (*reinterpret_cast<const volatile int*>(err) != 0) return false;
      const long long now = clock64();
      if (t0 == 0) t0 = now;
      else if (now - t0 > *reinterpret_cast<volatile long long*>(&g_wait_limit_cycles)) return false;
    }
  }
}

// column j of an output whose weight rows are interleaved in groups of 64 (first | second product)
__device__ __forceinline__ int sb_il(int j) { return (j >> 6) * 128 + (j & 63); }

// (mean, M2) over the 32 lanes of a warp, one value per lane
__device__ __forceinline__ void sb_warp_stats(float val, float& mean, float& m2) {
  float s = val;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  mean = s * (1.0f / 32.0f);
  const float d = val - mean;
  m2 = d * d;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m2 += __shfl_xor_sync(0xffffffffu, m2, o);
}

// The same for 16 values per lane at once (16 rows of one column): the 16 reductions of a level are independent, so
// their shuffles overlap instead of forming 16 chains of ten dependent ones.
__device__ __forceinline__ void sb_warp_stats16(const float* val, float* mean, float* m2) {
  float s[kSbGroup];
#pragma unroll
  for (int i = 0; i < kSbGroup; ++i) s[i] = val[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
    for (int i = 0; i < kSbGroup; ++i) s[i] += __shfl_xor_sync(0xffffffffu, s[i], o);
  }
#pragma unroll
  for (int i = 0; i < kSbGroup; ++i) { mean[i] = s[i] * (1.0f / 32.0f); const float d = val[i] - mean[i]; m2[i] = d * d; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
    for (int i = 0; i < kSbGroup; ++i) m2[i] += __shfl_xor_sync(0xffffffffu, m2[i], o);
  }
}

template <typename ACT, int AB_FMT>
__global__ void __launch_bounds__(kSbThreads, 1)
sb_chain_kernel(const __grid_constant__ CUtensorMap tmAp, const __grid_constant__ CUtensorMap tmV,
                const __grid_constant__ CUtensorMap tmS, const SbParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int W = p.W, L = p.L, T = p.T;
  const int kb_all = W / kBlockK;                // k-blocks of a product
  uint8_t* ring = smem;                          // dependent CTAs: 2 x 64 KB of weights; early CTAs: 6 x 32 KB
  uint8_t* bbuf = smem + kSbStages * kSbStageBytes;   // dependent CTAs: the group's activations
  uint8_t* misc = smem + (kSbDepBytes > kSbEarlyBytes ? kSbDepBytes : kSbEarlyBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(misc);          // up to 32 barriers
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(misc + 256);
  int* flag_s = reinterpret_cast<int*>(misc + 264);
  float* fs = reinterpret_cast<float*>(misc + 512);            // small float scratch (2.5 KB)
  const float** bias_s = reinterpret_cast<const float**>(misc + 3072);   // the bias pointer table (5 L + 2 <= 122 entries)

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rank = static_cast<int>(cluster_ctarank());
  const int cl = static_cast<int>(blockIdx.x) / kSbCluster;
  const bool is_dep = cl < p.nd;

  // dependent CTAs: full[2], empty[2], acc_full[2], b_full[6] (activations, one per 4 k-blocks)
  // early CTAs: full[6], empty[6], acc_full[2], acc_empty[2]
  uint64_t *d_full = bars, *d_empty = bars + kSbStages, *acc_full = bars + 2 * kSbStages, *b_full = bars + 2 * kSbStages + 2;
  uint64_t *e_full = bars, *e_empty = bars + kSbEarlyStages, *e_acc_full = bars + 2 * kSbEarlyStages,
           *e_acc_empty = bars + 2 * kSbEarlyStages + 2;
  if (tid == 0) {
    if (is_dep) {
      for (int s = 0; s < kSbStages; ++s) { mbar_init(&d_full[s], 1); mbar_init(&d_empty[s], 1); }
      for (int i = 0; i < kSbMaxW / (kBlockK * kSbKps); ++i) mbar_init(&b_full[i], 1);
      mbar_init(&acc_full[0], 1); mbar_init(&acc_full[1], 1);
    } else {
      for (int s = 0; s < kSbEarlyStages; ++s) { mbar_init(&e_full[s], 1); mbar_init(&e_empty[s], 1); }
      for (int i = 0; i < 2; ++i) { mbar_init(&e_acc_full[i], 1); mbar_init(&e_acc_empty[i], 1); }
    }
    fence_mbar_init();
    *flag_s = 1;
  }
  for (int i = tid; i < 5 * L + 2; i += kSbThreads) bias_s[i] = p.bias[i];
  if (warp == 1) { tmem_alloc(tmem_base_s, 256); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_base_s;
  const int NM = p.nm;
  const int nrep = p.cfg ? 2 : 1;

  if (is_dep) {
    // ================================================================== dependent chain of row group `cl`
    constexpr uint32_t idesc = umma_idesc_f16(kSbGroup, AB_FMT);
    const int grp = cl, row0 = grp * kSbGroup;
    const int ntile = W / 128;
    const int my_tiles = rank < ntile ? (ntile - rank + kSbCluster - 1) / kSbCluster : 0;   // column tiles rank, rank + 8
    const int wq = warp & 3;                     // worker warp's TMEM lane quarter
    const int wt = tid - 64;                     // worker index (warps 2..5)
    const int c = wq * 32 + lane;                // worker's column inside a tile (= TMEM lane)
    const int G = T * 2 * L;                     // product phases

    // Ends a phase: this CTA's global writes are published to the cluster, then the group's eight CTAs meet.
    auto cluster_sync_all = [&]() {
      if (warp >= 2) fence_proxy_async_all();    // the workers' generic-proxy writes, for the peers' TMA loads
      cluster_arrive();
      cluster_wait();
      if (warp == 0) fence_proxy_async_all();    // ... which this warp issues
    };

    // Step boundary, first half (token-parallel: one or two tokens of the group per CTA).  finish_t > 0: finish step
    // finish_t (final modulate, output projection, guidance, Eq. 3) and leave x_{t-1} in p.x; finish_t == 0: x <- x_T.
    auto finish_phase = [&](int finish_t) {
      if (warp < 2) return;
      float* eh = fs + 16;           // [2][16]
      float* rs = fs + 48;           // [2][2] mean, rstd
      float* part = fs + 64;         // [4 warps][2][16]
      const int per = p.cfg ? 8 : 16;            // tokens per group
      for (int q = rank; q < per; q += kSbCluster) {
        const int i = grp * per + q;             // token
        if (i >= p.R) break;
        const int rho0 = row0 + q, rho1 = row0 + 8 + q;    // its conditional / unconditional row (kernel order)
        if (finish_t == 0) {
          if (wt < p.C) p.x[static_cast<size_t>(i) * p.C + wt] = p.x_T[static_cast<size_t>(i) * p.C + wt];
          continue;
        }
        const float* mods = p.mods + static_cast<size_t>(finish_t & 1) * kSbRows * NM + 5 * L * W;
        if (wt < nrep) {
          float mean, rstd;
          row_stats<true>(p.stats, wt ? rho1 : rho0, W, mean, rstd);
          rs[wt * 2] = mean; rs[wt * 2 + 1] = rstd;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        float acc[2][kCPad];
#pragma unroll
        for (int e = 0; e < kCPad; ++e) { acc[0][e] = 0.0f; acc[1][e] = 0.0f; }
        for (int j0 = 0; j0 < W; j0 += 4 * kSbWorkers) {       // W is a multiple of 512: four columns per thread and turn
          float sh[2][4], scv[2][4], hv[2][4], bshv[4], bscv[4];
          float4 wv[4][4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int j = j0 + u * kSbWorkers + c;
            bshv[u] = bias_s[5 * L][j]; bscv[u] = bias_s[5 * L + 1][j];
#pragma unroll
            for (int rep = 0; rep < 2; ++rep) {
              if (rep < nrep) {
                const size_t row = rep ? rho1 : rho0;
                sh[rep][u] = __ldcg(mods + row * NM + sb_il(j)); scv[rep][u] = __ldcg(mods + row * NM + sb_il(j) + 64);
                hv[rep][u] = __ldcg(p.h + row * W + j);
              }
            }
            const float4* w4 = reinterpret_cast<const float4*>(p.wout_t + static_cast<size_t>(j) * kCPad);
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) wv[u][q4] = __ldg(w4 + q4);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float bsh = bshv[u], bsc = bscv[u];
#pragma unroll
            for (int rep = 0; rep < 2; ++rep) {
              if (rep < nrep) {
                const float uf = fmaf(__fmul_rn(__fsub_rn(hv[rep][u], rs[rep * 2]), rs[rep * 2 + 1]), __fadd_rn(1.0f, scv[rep][u] + bsc), sh[rep][u] + bsh);
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                  acc[rep][4 * q4] = fmaf(uf, wv[u][q4].x, acc[rep][4 * q4]); acc[rep][4 * q4 + 1] = fmaf(uf, wv[u][q4].y, acc[rep][4 * q4 + 1]);
                  acc[rep][4 * q4 + 2] = fmaf(uf, wv[u][q4].z, acc[rep][4 * q4 + 2]); acc[rep][4 * q4 + 3] = fmaf(uf, wv[u][q4].w, acc[rep][4 * q4 + 3]);
                }
              }
            }
          }
        }
#pragma unroll
        for (int rep = 0; rep < 2; ++rep) {
#pragma unroll
          for (int e = 0; e < kCPad; ++e) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc[rep][e] += __shfl_xor_sync(0xffffffffu, acc[rep][e], o);
          }
        }
        if (lane == 0) {
#pragma unroll
          for (int rep = 0; rep < 2; ++rep)
#pragma unroll
            for (int e = 0; e < kCPad; ++e) part[(wq * 2 + rep) * kCPad + e] = acc[rep][e];
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (wt < 2 * kCPad) {
          const int rep = wt >> 4, e = wt & 15;
          eh[wt] = ((part[(0 * 2 + rep) * kCPad + e] + part[(1 * 2 + rep) * kCPad + e]) + (part[(2 * 2 + rep) * kCPad + e] + part[(3 * 2 + rep) * kCPad + e])) + p.bout[e];
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (wt < p.C) {
          const size_t o = static_cast<size_t>(i) * p.C + wt;
          float e = eh[wt];
          if (p.cfg) e = cfg_combine(eh[wt], eh[kCPad + wt], p.cfg_scale);
          const float xo = __ldcg(p.x + o);
          const float mu = ddpm_mean(p.sched[finish_t - 1], xo, p.sched[T + finish_t - 1], e);
          const float xn = ddpm_sample(mu, p.sched[2 * T + finish_t - 1], p.eps[static_cast<size_t>(finish_t - 1) * p.R * p.C + o]);
          if (!(fabsf(xn) <= 3.0e38f)) *p.status = 1;
          if (finish_t == 1) {
            p.mu1[o] = mu;
            if (p.x1) p.x1[o] = xo;
            if (p.sample_last && p.x0) p.x0[o] = xn;
          } else p.x[o] = xn;
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
      }
    };
    // Step boundary, second half (column-parallel: this CTA's 128-column tiles for all rows of the group): input
    // projection h = Win x + bin, its LayerNorm partials, and a' = h (1 + scale) of block 0 with step prep_t's scale.
    auto prep_phase = [&](int prep_t) {
      if (warp < 2) return;
      float* xg = fs;                // [16 tokens][16] states of the group's tokens
      float* xch = fs + 256;         // [16 rows][4 warps][2]
      const int per = p.cfg ? 8 : 16;
      const float* mods = p.mods + static_cast<size_t>(prep_t & 1) * kSbRows * NM;
      for (int e = wt; e < per * kCPad; e += kSbWorkers) {
        const int tk = e >> 4, cc = e & 15, i = grp * per + tk;
        xg[e] = (i < p.R && cc < p.C) ? __ldcg(p.x + static_cast<size_t>(i) * p.C + cc) : 0.0f;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");
      for (int ti = 0; ti < my_tiles; ++ti) {
        const int tile = rank + ti * kSbCluster, col = tile * 128 + c;
        float sc[kSbGroup];
        const float* sp = mods + static_cast<size_t>(row0) * NM + 3 * W + sb_il(col) + 64;
#pragma unroll
        for (int i = 0; i < kSbGroup; ++i) sc[i] = __ldcg(sp + static_cast<size_t>(i) * NM);
        float wr[kCPad];
        const float4* w4 = reinterpret_cast<const float4*>(p.win + static_cast<size_t>(col) * kCPad);
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) { const float4 wv = __ldg(w4 + q4); wr[4 * q4] = wv.x; wr[4 * q4 + 1] = wv.y; wr[4 * q4 + 2] = wv.z; wr[4 * q4 + 3] = wv.w; }
        const float bi = p.bin[col], bs = bias_s[4][col];
        float* hout = p.h + static_cast<size_t>(row0) * W + col;
        ACT* aout = reinterpret_cast<ACT*>(p.ap) + static_cast<size_t>(row0) * W + col;
        float hv[kSbGroup], mean16[kSbGroup], m216[kSbGroup];
#pragma unroll
        for (int i = 0; i < kSbGroup; ++i) {
          const int tk = p.cfg ? (i & 7) : i;    // the row's token within the group (both guidance rows share x)
          const float4* xq = reinterpret_cast<const float4*>(xg + tk * kCPad);
          float a = bi;
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const float4 xv = xq[q4];
            a = fmaf(wr[4 * q4], xv.x, a); a = fmaf(wr[4 * q4 + 1], xv.y, a); a = fmaf(wr[4 * q4 + 2], xv.z, a); a = fmaf(wr[4 * q4 + 3], xv.w, a);
          }
          hv[i] = a;
        }
#pragma unroll
        for (int i = 0; i < kSbGroup; ++i) {
          hout[static_cast<size_t>(i) * W] = hv[i];
          aout[static_cast<size_t>(i) * W] = to_act<ACT>(__fmul_rn(hv[i], __fadd_rn(1.0f, __fadd_rn(sc[i], bs))));
        }
        sb_warp_stats16(hv, mean16, m216);
        if (lane == 0) {
#pragma unroll
          for (int i = 0; i < kSbGroup; ++i) { xch[(i * 4 + wq) * 2] = mean16[i]; xch[(i * 4 + wq) * 2 + 1] = m216[i]; }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (wt < 2 * kSbGroup) {
          const int i = wt >> 1, pr = (wt & 1) * 2;
          float pm = xch[(i * 4 + pr) * 2], pm2 = xch[(i * 4 + pr) * 2 + 1];
          chan_merge_equal(pm, pm2, xch[(i * 4 + pr + 1) * 2], xch[(i * 4 + pr + 1) * 2 + 1], 32.0f);
          reinterpret_cast<float2*>(p.stats)[static_cast<size_t>(row0 + i) * (W / kStatCols) + tile * 2 + (wt & 1)] = make_float2(pm, pm2);
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
      }
    };
    // one thread waits for the early products of step t
    auto wait_mods = [&](int t) {
      if (tid == 64 && !sb_wait_count(&p.sync[1 + t], p.ntasks, p.err)) ch_fail(p.err, 3, 9, t);
      asm volatile("bar.sync 1, 128;" ::: "memory");
    };

    // weight stream of this CTA: phase g, tile ti, stage of 4 k-blocks  ->  ring slot (running index % stages)
    const int sps = kb_all / kSbKps;             // stages per tile and phase
    const int stages_per_phase = my_tiles * sps;
    int issued = 0;                              // TMA warp: stages requested so far
    auto stream_weights = [&](int upto) {        // one lane: request stages while issued < upto
      while (issued < upto && issued < G * stages_per_phase) {
        const int g = issued / stages_per_phase, rem = issued % stages_per_phase;
        const int ti = rem / sps, kb0 = (rem % sps) * kSbKps;
        const int s = issued % kSbStages;
        if (issued >= kSbStages && !ch_wait<false>(&d_empty[s], ((issued / kSbStages) & 1) ^ 1, p.err)) { ch_fail(p.err, 1, 10, issued); return; }
        mbar_arrive_expect_tx(&d_full[s], kSbStageBytes);
#pragma unroll
        for (int j = 0; j < kSbKps; ++j)
          tma_load_2d(ring + s * kSbStageBytes + j * 16384, p.maps + (g % (2 * L)), &d_full[s], (kb0 + j) * kBlockK, (rank + ti * kSbCluster) * 128);
        ++issued;
      }
    };

    // ---- start: the weight ring fills while the first step's early products are awaited
    cluster_arrive(); cluster_wait();
    if (warp == 0 && lane == 0 && my_tiles > 0) stream_weights(kSbStages);
    finish_phase(0);
    cluster_sync_all();
    if (warp >= 2) wait_mods(T);
    prep_phase(T);
    cluster_sync_all();

    int g = 0, consumed = 0;                     // MMA warp: blocks consumed
    for (int t = T; t >= 1; --t) {
      const float* mods = p.mods + static_cast<size_t>(t & 1) * kSbRows * NM;
      for (int ph = 0; ph < 2 * L; ++ph, ++g) {
        const int k = ph >> 1;
        const bool second = (ph & 1) != 0;       // W2 product (gate + residual) or W1 product (folded LayerNorm + SiLU)
        if (warp == 0) {
          if (my_tiles > 0) {
            // the group's activations of this phase (written by the cluster before the barrier just passed), four
            // k-blocks (8 KB) per barrier so that the first MMAs need not wait for all of them
            if (lane < sps) mbar_arrive_expect_tx(&b_full[lane], kSbKps * kSbGroup * 128);
            __syncwarp();
            const CUtensorMap* m = second ? &tmV : &tmAp;
            for (int kb = lane; kb < kb_all; kb += 32) tma_load_2d(bbuf + kb * (kSbGroup * 128), m, &b_full[kb / kSbKps], kb * kBlockK, row0);
            // rest of this phase's weights, then as much of the next phase's as the ring holds
            if (lane == 0) stream_weights((g + 1) * stages_per_phase + kSbStages);
          }
          __syncwarp();
        } else if (warp == 1) {
          if (my_tiles > 0) {
            bool w_ok = true;
            const uint64_t db0 = umma_smem_desc_sw128(smem_u32(bbuf));
            for (int ti = 0; ti < my_tiles; ++ti) {
              for (int sg = 0; sg < sps; ++sg, ++consumed) {
                const int s = consumed % kSbStages;
                if (w_ok && ti == 0 && !ch_wait<false>(&b_full[sg], g & 1, p.err)) { if (lane == 0) ch_fail(p.err, 2, 11, g); w_ok = false; }
                if (w_ok && !ch_wait<false>(&d_full[s], (consumed / kSbStages) & 1, p.err)) { if (lane == 0) ch_fail(p.err, 2, 12, consumed); w_ok = false; }
                if (w_ok) {
                  tc_fence_after_sync();
                  if (elect_one()) {
                    const uint64_t da0 = umma_smem_desc_sw128(smem_u32(ring + s * kSbStageBytes));
#pragma unroll
                    for (int j = 0; j < kSbKps; ++j) {
                      const uint64_t da = da0 + static_cast<uint64_t>(j * (16384 >> 4));
                      const uint64_t db = db0 + static_cast<uint64_t>((sg * kSbKps + j) * ((kSbGroup * 128) >> 4));
#pragma unroll
                      for (int kk = 0; kk < kBlockK / 16; ++kk) umma_f16(tmem_base + ti * 32, da + 2 * kk, db + 2 * kk, idesc, (sg > 0 || j > 0 || kk > 0) ? 1u : 0u);
                    }
                    umma_commit(&d_empty[s]);
                  }
                  __syncwarp();
                }
              }
              if (w_ok && elect_one()) umma_commit(&acc_full[ti]);
              __syncwarp();
            }
          }
        } else {
          // ---- workers: everything the epilogue needs that is already in memory is fetched while the product runs
          float* rsm = fs;             // [16][2] mean, rstd of the group's rows
          float* xch = fs + 64;        // [16 rows][4 warps][2]
          if (!second) {
            if (wt < kSbGroup) {
              // (rows of the group beyond the call's hold whatever the buffers hold: computed, stored, never used)
              float mean, rstd;
              row_stats<true>(p.stats, row0 + wt, W, mean, rstd);
              rsm[wt * 2] = mean; rsm[wt * 2 + 1] = rstd;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
          }
          for (int ti = 0; ti < my_tiles; ++ti) {
            const int tile = rank + ti * kSbCluster, col = tile * 128 + c;
            const float* const* bb = bias_s + 5 * k;
            float m0[kSbGroup], m1[kSbGroup], hv[kSbGroup];
            // this column's constants: first layer c1, c2; second layer gate bias, b2, next block's scale bias
            const float kb0 = second ? bb[2][col] : bb[0][col], kb1 = second ? bb[3][col] : bb[1][col];
            const float kb2 = (second && k + 1 < L) ? bias_s[5 * (k + 1) + 4][col] : 0.0f;
            if (!second) {
              const float* mp = mods + static_cast<size_t>(row0) * NM + 5 * k * W + sb_il(col);
#pragma unroll
              for (int i = 0; i < kSbGroup; ++i) { m0[i] = __ldcg(mp + static_cast<size_t>(i) * NM); m1[i] = __ldcg(mp + static_cast<size_t>(i) * NM + 64); }
            } else {
              const float* gp = mods + static_cast<size_t>(row0) * NM + 5 * k * W + 2 * W + col;
              const float* sp = mods + static_cast<size_t>(row0) * NM + 5 * (k + 1) * W + 3 * W + sb_il(col) + 64;   // next block's scale
#pragma unroll
              for (int i = 0; i < kSbGroup; ++i) {
                m0[i] = __ldcg(gp + static_cast<size_t>(i) * NM);
                m1[i] = (k + 1 < L) ? __ldcg(sp + static_cast<size_t>(i) * NM) : 0.0f;
                hv[i] = __ldcg(p.h + static_cast<size_t>(row0 + i) * W + col);
              }
            }
            bool w_ok = true;
            if (lane == 0) w_ok = ch_wait<false>(&acc_full[ti], g & 1, p.err);
            w_ok = __shfl_sync(0xffffffffu, w_ok ? 1 : 0, 0) != 0;
            if (!w_ok && lane == 0) ch_fail(p.err, 3, 13, g);     // (the barriers below are still taken)
            tc_fence_after_sync();
            float acc[kSbGroup];
            tmem_ld16(tmem_base + (static_cast<uint32_t>(wq * 32) << 16) + ti * 32, acc);
            tmem_ld_wait();
            tc_fence_before_sync();
            if (!second) {
              const float k1 = kb0, k2 = kb1;
              ACT* vout = reinterpret_cast<ACT*>(p.v) + static_cast<size_t>(row0) * W + col;
#pragma unroll
              for (int i = 0; i < kSbGroup; ++i) {
                const float t1 = __fsub_rn(acc[i], __fmul_rn(rsm[i * 2], __fadd_rn(m0[i], k1)));
                vout[static_cast<size_t>(i) * W] = to_act<ACT>(silu_t<true>(fmaf(rsm[i * 2 + 1], t1, __fadd_rn(m1[i], k2))));
              }
            } else {
              const float bg = kb0, b2 = kb1, bsn = kb2;
              float* hout = p.h + static_cast<size_t>(row0) * W + col;
              ACT* aout = reinterpret_cast<ACT*>(p.ap) + static_cast<size_t>(row0) * W + col;
#pragma unroll
              for (int i = 0; i < kSbGroup; ++i) {
                hv[i] = fmaf(__fadd_rn(m0[i], bg), __fadd_rn(acc[i], b2), hv[i]);
                hout[static_cast<size_t>(i) * W] = hv[i];
                if (k + 1 < L) aout[static_cast<size_t>(i) * W] = to_act<ACT>(__fmul_rn(hv[i], __fadd_rn(1.0f, __fadd_rn(m1[i], bsn))));
              }
              // LayerNorm partials of the new h: (mean, M2) per row and 64-column group (two warps)
              float mean16[kSbGroup], m216[kSbGroup];
              sb_warp_stats16(hv, mean16, m216);
              if (lane == 0) {
#pragma unroll
                for (int i = 0; i < kSbGroup; ++i) { xch[(i * 4 + wq) * 2] = mean16[i]; xch[(i * 4 + wq) * 2 + 1] = m216[i]; }
              }
              asm volatile("bar.sync 1, 128;" ::: "memory");
              if (wt < 2 * kSbGroup) {
                const int i = wt >> 1, pr = (wt & 1) * 2;
                float pm = xch[(i * 4 + pr) * 2], pm2 = xch[(i * 4 + pr) * 2 + 1];
                chan_merge_equal(pm, pm2, xch[(i * 4 + pr + 1) * 2], xch[(i * 4 + pr + 1) * 2 + 1], 32.0f);
                reinterpret_cast<float2*>(p.stats)[static_cast<size_t>(row0 + i) * (W / kStatCols) + tile * 2 + (wt & 1)] = make_float2(pm, pm2);
              }
              asm volatile("bar.sync 1, 128;" ::: "memory");
            }
          }
        }
        cluster_sync_all();
      }
      // ---- step boundary: finish step t, prepare step t - 1 (its early products must be complete)
      finish_phase(t);
      cluster_sync_all();
      if (t > 1) {
        if (warp >= 2) wait_mods(t - 1);
        prep_phase(t - 1);
        cluster_sync_all();
      }
      if (rank == 0 && tid == 0) { __threadfence(); atomicAdd(&p.sync[0], 1); }    // this group is done with the slot of step t
    }
  } else {
    // ================================================================== early products of s_t
    constexpr uint32_t idesc = umma_idesc_f16(kSbRows, AB_FMT);
    const int ecta = (cl - p.nd) * kSbCluster + rank, nec = p.ne * kSbCluster;
    const int wq = warp & 3;
    const int c = wq * 32 + lane;
    bool ok = true;
    if (warp == 0) {
      int it = 0;
      for (int t = T; t >= 1 && ok; --t) {
        // the slot of step t was last read in step t + 2: wait until every row group has finished that step
        if (t + 2 <= T) {
          int good = 1;
          if (lane == 0 && !sb_wait_count(&p.sync[0], (T - (t + 2) + 1) * p.nd, p.err)) { ch_fail(p.err, 1, 14, t); good = 0; }
          good = __shfl_sync(0xffffffffu, good, 0);
          if (!good) { ok = false; break; }
        }
        for (int j = ecta; j < p.ntasks && ok; j += nec) {
          const SbTask task = p.tasks[j];
          for (int kb = 0; kb < kb_all; ++kb, ++it) {
            const int s = it % kSbEarlyStages;
            int good = 1;
            if (lane == 0) {
              if (it >= kSbEarlyStages && !ch_wait<false>(&e_empty[s], ((it / kSbEarlyStages) & 1) ^ 1, p.err)) { ch_fail(p.err, 1, 15, it); good = 0; }
              if (good) {
                mbar_arrive_expect_tx(&e_full[s], 32768);
                tma_load_2d(ring + s * 32768, p.maps + task.map, &e_full[s], kb * kBlockK, task.row);
                tma_load_2d(ring + s * 32768 + 16384, &tmS, &e_full[s], kb * kBlockK, (t - 1) * kSbRows);
              }
            }
            good = __shfl_sync(0xffffffffu, good, 0);
            if (!good) { ok = false; break; }
          }
        }
      }
    } else if (warp == 1) {
      int it = 0, n = 0;
      for (int t = T; t >= 1 && ok; --t) {
        for (int j = ecta; j < p.ntasks && ok; j += nec, ++n) {
          const int ab = n & 1;
          if (n >= 2 && !ch_wait<false>(&e_acc_empty[ab], ((n >> 1) - 1) & 1, p.err)) { if (lane == 0) ch_fail(p.err, 2, 16, n); ok = false; break; }
          tc_fence_after_sync();
          for (int kb = 0; kb < kb_all; ++kb, ++it) {
            const int s = it % kSbEarlyStages;
            if (!ch_wait<false>(&e_full[s], (it / kSbEarlyStages) & 1, p.err)) { if (lane == 0) ch_fail(p.err, 2, 17, it); ok = false; break; }
            tc_fence_after_sync();
            if (elect_one()) {
              const uint32_t sa = smem_u32(ring + s * 32768);
              const uint64_t da = umma_smem_desc_sw128(sa), db = umma_smem_desc_sw128(sa + 16384);
#pragma unroll
              for (int kk = 0; kk < kBlockK / 16; ++kk) umma_f16(tmem_base + ab * kSbRows, da + 2 * kk, db + 2 * kk, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
              umma_commit(&e_empty[s]);
            }
            __syncwarp();
          }
          if (ok && elect_one()) umma_commit(&e_acc_full[ab]);
          __syncwarp();
        }
      }
    } else {
      int n = 0;
      // rows (kernel order) that belong to the call, as a 128-bit mask in four words
      uint32_t valid[4] = {0u, 0u, 0u, 0u};
      for (int rho = 0; rho < kSbRows; ++rho) { int rep; if (sb_row_token(rho, p.cfg, &rep) < p.R) valid[rho >> 5] |= 1u << (rho & 31); }
      for (int t = T; t >= 1 && ok; --t) {
        float* mods = p.mods + static_cast<size_t>(t & 1) * kSbRows * NM;
        int done = 0;
        for (int j = ecta; j < p.ntasks && ok; j += nec, ++n, ++done) {
          const SbTask task = p.tasks[j];
          const int ab = n & 1;
          int good = 1;
          if (lane == 0 && !ch_wait<false>(&e_acc_full[ab], (n >> 1) & 1, p.err)) { ch_fail(p.err, 3, 18, n); good = 0; }
          good = __shfl_sync(0xffffffffu, good, 0);
          if (!good) { ok = false; break; }
          tc_fence_after_sync();
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            float a[kChunk];
            tmem_ld32(tmem_base + (static_cast<uint32_t>(wq * 32) << 16) + ab * kSbRows + ch * kChunk, a);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < kChunk; ++i)
              if ((valid[ch] >> i) & 1u) mods[static_cast<size_t>(ch * kChunk + i) * NM + task.col + c] = a[i];
          }
          tc_fence_before_sync();
          asm volatile("bar.sync 1, 128;" ::: "memory");
          if (tid == 64) mbar_arrive(&e_acc_empty[ab]);
        }
        // this CTA's tiles of step t are in global memory
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (tid == 64 && ok && done > 0) atomicAdd(&p.sync[1 + t], done);
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, 256);
}

// s_t = SiLU(cz + te_t) for every step at once, in operand format and in the kernel's row order, one 128-row block
// per step (the early products' B operand): s_all[(t - 1) * 128 + rho][col].
template <typename ACT>
__global__ void __launch_bounds__(256) sb_cond_all_kernel(const float* __restrict__ cz, const float* __restrict__ te,
                                                          ACT* __restrict__ s_all, int R, int cfg, int W, int T) {
  const int t = blockIdx.y, rho = blockIdx.x;
  int rep;
  const int i = sb_row_token(rho, cfg, &rep);
  if (i >= R) return;
  const size_t src = static_cast<size_t>(rep) * R + i;
  for (int j = threadIdx.x; j < W; j += blockDim.x)
    s_all[(static_cast<size_t>(t) * kSbRows + rho) * W + j] = to_act<ACT>(silu_f(cz[src * W + j] + te[static_cast<size_t>(t) * W + j]));
}

}  // namespace csd
