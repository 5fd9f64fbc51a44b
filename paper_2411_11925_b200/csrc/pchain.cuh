// One persistent kernel per chain for layers of one wave (W = 1024, a few hundred to a few thousand head rows).
//
// With one kernel per layer a chain is a sequence of dependent launches: each waits for the whole preceding grid, and
// the early part of the next kernel has to find free SMs beside it.  Two chains side by side (draft and target of a
// round) ask for twice the SMs the GPU has, so their kernels start piecemeal.  Here a CTA owns one 128 x 128 output
// tile of EVERY layer for ALL denoising steps:
//   * rows never exchange data in a per-token MLP, so the only synchronisation is between the CTAs that share rows:
//     the 8 column tiles of a row block (and, because two row blocks share each MMA as a CTA pair, the 16 CTAs of two
//     row blocks).  They meet at a counter in global memory once per layer; different groups never wait for each other,
//     so nothing requires the whole grid to be resident.
//   * the products that depend only on the condition vector s_t (gate, scales, the folded P1 | P2) are issued by the
//     same CTA into TMEM before the product that waits for its neighbours, so the tensor pipe works while the
//     neighbours finish; their operands stream through the same ring.
//   * the residual stream h lives in TMEM (128 columns) for the whole chain: it is read and written only by the tile's
//     own epilogues.  Activations (a', v: 16-bit) go through global memory / L2 by TMA; LayerNorm partials, the
//     output-projection partials and the token states x_t through plain global memory.
// All blocks run in the folded form of fold.cuh (block 0 too): phases per step
//   B     : early [shift_0 | scale_0] = s Wss_0^T;  h = Win x + bin, LayerNorm partials, a' = h (1 + scale_0)
//   W1_k  : early [P1 | P2];  dependent a' W1_k^T;  v = SiLU(rstd (acc - mean (P1 + c1)) + P2 + c2)
//   GATE_k: early [gate_k | scale_{k+1}] (last block: gate only);  dependent v W2_k^T;  h += gate (acc + b2), partials,
//           a' = h (1 + scale_{k+1})
//   F     : early [shift_f | scale_f];  eps partial = (LN(h)(1 + scale_f) + shift_f) Wout^T tile
//   U     : (token-parallel, between steps) eps reduction, guidance, Eq. 3 update of x.
// s_t of every step is precomputed (pc_cond_all_kernel) in the kernel's row order: a row block holds 64 tokens'
// conditional rows followed by their unconditional twins (128 tokens without guidance).
#pragma once
#include "fold.cuh"

namespace csd {

constexpr int kPcThreads = 384;            // TMA activations, MMA, 8 epilogue warps, TMA weights, TMA activations (2nd k-block)
constexpr int kPcGran = 16384;             // ring granule: one 128-row x 64-column 16-bit box
constexpr int kPcNG = 10;                  // granules in the ring (160 KB)
constexpr int kPcBars = 8;                 // full / empty barrier slots (at most 5 stages are in flight)
constexpr int kPcColTiles = 8;             // W / 128
constexpr int kPcGroup = 2 * kPcColTiles;  // CTAs that meet at a counter: two row blocks x 8 column tiles
constexpr uint32_t kPcAccP = 0, kPcAccM = 256, kPcAccH = 384;   // TMEM columns: packed early products, dependent product, h

constexpr int kPcRing = kPcNG * kPcGran;
constexpr int kPcOffStage = kPcRing;                       // 32 KB: 16-bit output tile on its way out
constexpr int kPcOffWin = kPcOffStage + 32768;             // [128 columns][16] fp32
constexpr int kPcOffWout = kPcOffWin + 8192;               // [128 columns][16] fp32
constexpr int kPcOffX = kPcOffWout + 8192;                 // [128 tokens][16] fp32
constexpr int kPcOffBias = kPcOffX + 8192;                 // [2][3][128] fp32
constexpr int kPcOffBin = kPcOffBias + 3072;               // [128]
constexpr int kPcOffEh = kPcOffBin + 512;                  // [256] eps sums of the update phase
constexpr int kPcOffBars = kPcOffEh + 1024;                // full[8], empty[8], acc_full[2], acc_empty, flags
constexpr int kPcSmemBytes = 1024 + kPcOffBars + 256;
static_assert(kPcSmemBytes <= 227 * 1024, "shared memory budget");

struct PcParams {
  int R, cfg, W, L, T, C, sample_last, nblk;   // nblk: row blocks of 128 kernel rows (even)
  float cfg_scale;
  const CUtensorMap* maps;     // [2 (2L + 2)]: per phase the early weights, then per phase the dependent weights
  const float* const* bias;    // [2L + 2][3]
  const float* sched;          // a[T], b[T], sigma[T]
  const float *win, *bin, *wout_t, *bout;
  const float *x_T, *eps;
  float *x0, *mu1, *x1;
  float *traj_x, *traj_mu;     // optional records: slot j of traj_x holds x_{T-j} ([T+1, R, C]), of traj_mu mu_{T-j} ([T, R, C])
  float* x;                    // [R, C] state between steps
  float* stats;                // [nblk 128, W/64, 2]
  float* epart;                // [nblk 128, W/64, 16]
  unsigned* sync;              // [nblk / 2] arrivals
  int* err;
  int* status;
};

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float* v) {
  const uint32_t* r = reinterpret_cast<const uint32_t*>(v);
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]),
        "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]),
        "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ unsigned pc_ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void pc_arrive(unsigned* p) {
  asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}
// One thread waits until the counter has reached target (bounded; gives up once the context's status word is up).
__device__ __forceinline__ bool pc_wait_count(const unsigned* p, unsigned target, const int* err) {
  long long t0 = 0;
  uint32_t spins = 0;
  for (;;) {
    if (pc_ld_acquire(p) >= target) return true;
    __nanosleep(40);   // the poll is a round trip to L2 anyway; idle issue slots instead of a hot loop (the GPU runs at its power cap)
    if ((++spins & 255u) == 0u) {
      if (*reinterpret_cast<const volatile int*>(err) != 0) return false;
      const long long now = clock64();
      if (t0 == 0) t0 = now;
      else if (now - t0 > *reinterpret_cast<volatile long long*>(&g_wait_limit_cycles)) return false;
    }
  }
}

__device__ __forceinline__ void pc_flag_set(uint32_t* smem_word, uint32_t v) {
  asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(smem_u32(smem_word)), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t pc_flag_get(const uint32_t* smem_word) {
  uint32_t v;
  asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(smem_word)) : "memory");
  return v;
}
// One thread waits until this CTA's flag word has reached target (bounded).
__device__ __forceinline__ bool pc_wait_flag(const uint32_t* smem_word, uint32_t target, const int* err) {
  long long t0 = 0;
  uint32_t spins = 0;
  for (;;) {
    if (pc_flag_get(smem_word) >= target) return true;
    if ((++spins & 1023u) == 0u) {
      if (*reinterpret_cast<const volatile int*>(err) != 0) return false;
      const long long now = clock64();
      if (t0 == 0) t0 = now;
      else if (now - t0 > *reinterpret_cast<volatile long long*>(&g_wait_limit_cycles)) return false;
    }
  }
}

// Token and guidance row (0 conditional, 1 unconditional) of kernel row rho.
__host__ __device__ __forceinline__ int pc_row_token(int rho, int cfg, int* rep) {
  const int blk = rho >> 7, r = rho & 127;
  if (!cfg) { *rep = 0; return blk * 128 + r; }
  *rep = r >> 6;
  return blk * 64 + (r & 63);
}

template <typename ACT, int AB_FMT>
__global__ void __launch_bounds__(kPcThreads, 1)
pchain_kernel(const __grid_constant__ CUtensorMap tmS, const __grid_constant__ CUtensorMap tmAp,
              const __grid_constant__ CUtensorMap tmV, const PcParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* ring = smem;
  uint8_t* stage_out = smem + kPcOffStage;
  float* win_s = reinterpret_cast<float*>(smem + kPcOffWin);
  float* wout_s = reinterpret_cast<float*>(smem + kPcOffWout);
  float* xg = reinterpret_cast<float*>(smem + kPcOffX);
  float* bias_all = reinterpret_cast<float*>(smem + kPcOffBias);
  float* bin_s = reinterpret_cast<float*>(smem + kPcOffBin);
  float* eh = reinterpret_cast<float*>(smem + kPcOffEh);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kPcOffBars);
  uint64_t* empty_bar = full_bar + kPcBars;
  uint64_t* acc_full = empty_bar + kPcBars;     // [2]: packed, dependent
  uint64_t* acc_empty = acc_full + 2;           // the epilogues of both CTAs have read the accumulators
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(acc_empty + 1);
  volatile int* epi_ok_s = reinterpret_cast<volatile int*>(tmem_base_s + 1);
  uint32_t* meet_seen_s = tmem_base_s + 2;      // meeting points this CTA's epilogue has seen complete (count)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int W = p.W, L = p.L, T = p.T, nkb = W / kBlockK;
  const int NP = 2 * L + 2, NS = NP + 1;           // phases and meeting points per step
  const int rank = static_cast<int>(cluster_ctarank());
  const int cl = static_cast<int>(blockIdx.x >> 1);
  const int grp = cl / kPcColTiles, tile_n = cl % kPcColTiles, tile_m = 2 * grp + rank;
  const int n_base = tile_n * kTileN, row0 = tile_m * kTileM;
  const int rows_all = p.nblk * kTileM;
  unsigned* const ctr = p.sync + grp;

  const bool run = *reinterpret_cast<const volatile int*>(p.err) == 0;
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmS); tma_prefetch_desc(&tmAp); tma_prefetch_desc(&tmV);
    for (int s = 0; s < kPcBars; ++s) { mbar_init(&full_bar[s], 3); mbar_init(&empty_bar[s], 1); }
    mbar_init(&acc_full[0], 1); mbar_init(&acc_full[1], 1); mbar_init(acc_empty, 16);   // 8 epilogue warps of each CTA
    *epi_ok_s = 1;
    *meet_seen_s = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc_pair(tmem_base_s, 512); tmem_relinquish_pair(); }
  // constants of this column tile
  for (int i = threadIdx.x; i < kTileN * kCPad; i += kPcThreads) {
    win_s[i] = p.win[static_cast<size_t>(n_base) * kCPad + i];
    wout_s[i] = p.wout_t[static_cast<size_t>(n_base) * kCPad + i];
  }
  if (threadIdx.x < kTileN) bin_s[threadIdx.x] = p.bin[n_base + threadIdx.x];
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive(); cluster_wait();   // the peer's barriers exist before anything signals them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_base_s;

  auto has_dep = [&](int ph) { return ph != 0 && ph != NP - 1; };
  auto early_n128 = [&](int ph) { return ph == 2 * L; };      // last block's gate: a single product

  if (run && (warp == 0 || warp >= 10)) {
    // ------------------------------------------------------------------ TMA requests
    const bool is_a = warp != 10;
    const bool second = warp == 11;
    const bool leader = elect_one();
    bool ok = true;
    // head of the granule ring (stage count, position, absolute granule count) and the oldest stage not yet known free
    uint32_t n = 0, gpos = 0;
    int gabs = 0;
    uint32_t tn = 0;
    int tabs = 0, tph = 0, tpart = 0, tidx = 0;
    auto acquire = [&](int g) {          // make room for a stage of g granules
      while (ok && tabs < gabs + g - kPcNG) {
        ok = ch_wait<false>(&empty_bar[tn & (kPcBars - 1)], (tn / kPcBars) & 1, p.err);
        if (!ok) { if (leader) ch_fail(p.err, DEV_ERR_TMA_WAIT, 2, static_cast<int>(tn)); break; }
        tabs += tpart ? 3 : 2; ++tn; ++tidx;
        if (tpart == 0) { if (tidx == nkb) { tidx = 0; if (has_dep(tph)) tpart = 1; else tph = tph + 1 == NP ? 0 : tph + 1; } }
        else if (tidx == nkb / 2) { tidx = 0; tpart = 0; tph = tph + 1 == NP ? 0 : tph + 1; }
      }
    };
    auto gran = [&](int i) { uint32_t g = gpos + i; if (g >= kPcNG) g -= kPcNG; return ring + g * kPcGran; };
    auto advance = [&](int g) { ++n; gabs += g; gpos += g; if (gpos >= kPcNG) gpos -= kPcNG; };
    // A pair's loads are all credited to the leader's barrier, which only the leader's producers arm (with the bytes
    // of both CTAs); the peer's producers only request.
    auto arm = [&](uint64_t* bar, uint32_t bytes) { if (rank == 0) mbar_arrive_expect_tx(bar, 2 * bytes); };
    auto load = [&](uint8_t* dst, const CUtensorMap* tm, uint64_t* bar, int x, int y) {
      tma_load_2d_pair(dst, tm, mapa_shared(smem_u32(bar), 0), x, y);
    };
    for (int si = 0; si < T && ok; ++si) {
      const int t = T - si;
      const int srow = (t - 1) * rows_all + row0;
      for (int ph = 0; ph < NP && ok; ++ph) {
        const CUtensorMap* tmE = p.maps + ph;
        const bool n128 = early_n128(ph);
        // A dependent operand is complete once every CTA of the group has finished the preceding phase; this CTA's
        // epilogue watches the group's counter and raises a flag in shared memory.  The proxy fence that must follow
        // is taken between early stages as soon as the flag is up, off the path of the first dependent load.
        const uint32_t meet_target = static_cast<uint32_t>(si * NS + ph + 1);
        bool fenced = !(is_a && has_dep(ph));
        for (int kb = 0; kb < nkb && ok; ++kb) {
          acquire(2);
          if (ok && leader) {
            if (!fenced && kb >= nkb - 6 && pc_flag_get(meet_seen_s) >= meet_target) { fence_proxy_async_all(); fenced = true; }
            uint64_t* fb = &full_bar[n & (kPcBars - 1)];
            if (second) { if (rank == 0) mbar_arrive(fb); }
            else if (is_a) { arm(fb, 16384); load(gran(0), &tmS, fb, kb * kBlockK, srow); }
            else {
              arm(fb, n128 ? 8192 : 16384);
              load(gran(1), tmE, fb, kb * kBlockK, n128 ? n_base + rank * 64 : 2 * n_base + rank * 128);
            }
          }
          __syncwarp();
          advance(2);
        }
        if (!has_dep(ph)) continue;
        if (is_a && ok) {
          if (leader && !fenced) {
            if (!pc_wait_flag(meet_seen_s, meet_target, p.err)) { ch_fail(p.err, DEV_ERR_TMA_WAIT, 3, ph); ok = false; }
            fence_proxy_async_all();
          }
          ok = __all_sync(0xffffffffu, ok);
        }
        const CUtensorMap* tmA = (ph & 1) ? &tmAp : &tmV;      // W1 phases read a', GATE phases v
        const CUtensorMap* tmW = p.maps + NP + ph;
        for (int kb = 0; kb < nkb && ok; kb += 2) {
          acquire(3);
          if (ok && leader) {
            uint64_t* fb = &full_bar[n & (kPcBars - 1)];
            if (is_a) {
              const int jj = second ? 1 : 0;
              arm(fb, 16384);
              load(gran(jj), tmA, fb, (kb + jj) * kBlockK, row0);
            } else {
              arm(fb, 16384);
#pragma unroll
              for (int jj = 0; jj < 2; ++jj) load(gran(2) + jj * 8192, tmW, fb, (kb + jj) * kBlockK, n_base + rank * 64);
            }
          }
          __syncwarp();
          advance(3);
        }
      }
    }
  } else if (run && warp == 1 && rank == 0) {
    // ------------------------------------------------------------------ MMA issue (the pair's leader)
    const bool leader = elect_one();
    constexpr uint32_t idesc128 = umma_idesc_f16(128, AB_FMT, 256), idesc256 = umma_idesc_f16(256, AB_FMT, 256);
    bool ok = true;
    uint32_t n = 0, gpos = 0;
    int gp = 0;
    auto gaddr = [&](int i) { uint32_t g = gpos + i; if (g >= kPcNG) g -= kPcNG; return smem_u32(ring + g * kPcGran); };
    for (int si = 0; si < T && ok; ++si) {
      for (int ph = 0; ph < NP && ok; ++ph, ++gp) {
        if (gp > 0) {
          ok = ch_wait<true>(acc_empty, (gp - 1) & 1, p.err);
          if (!ok) { if (leader) ch_fail(p.err, DEV_ERR_MMA_WAIT, 5, gp); break; }
        }
        tc_fence_after_sync();
        const uint32_t idesc_e = early_n128(ph) ? idesc128 : idesc256;
        for (int kb = 0; kb < nkb && ok; ++kb) {
          const uint32_t slot = n & (kPcBars - 1);
          ok = ch_wait<false>(&full_bar[slot], (n / kPcBars) & 1, p.err);
          if (!ok) { if (leader) ch_fail(p.err, DEV_ERR_MMA_WAIT, 7, ph); break; }
          tc_fence_after_sync();
          if (leader) {
            const uint64_t da = umma_smem_desc_sw128(gaddr(0)), db = umma_smem_desc_sw128(gaddr(1));
#pragma unroll
            for (int k = 0; k < kBlockK / 16; ++k) umma_f16_pair(tmem_base + kPcAccP, da + 2 * k, db + 2 * k, idesc_e, (kb > 0 || k > 0) ? 1u : 0u);
            umma_commit_pair(&empty_bar[slot]);
          }
          __syncwarp();
          ++n; gpos += 2; if (gpos >= kPcNG) gpos -= kPcNG;
        }
        if (ok && leader) umma_commit_pair(&acc_full[0]);
        __syncwarp();
        if (!has_dep(ph)) continue;
        for (int kb = 0; kb < nkb && ok; kb += 2) {
          const uint32_t slot = n & (kPcBars - 1);
          ok = ch_wait<false>(&full_bar[slot], (n / kPcBars) & 1, p.err);
          if (!ok) { if (leader) ch_fail(p.err, DEV_ERR_MMA_WAIT, 6, ph); break; }
          tc_fence_after_sync();
          if (leader) {
            const uint32_t wb = gaddr(2);
#pragma unroll
            for (int jj = 0; jj < 2; ++jj) {
              const uint64_t da = umma_smem_desc_sw128(gaddr(jj)), db = umma_smem_desc_sw128(wb + jj * 8192);
#pragma unroll
              for (int k = 0; k < kBlockK / 16; ++k) umma_f16_pair(tmem_base + kPcAccM, da + 2 * k, db + 2 * k, idesc128, (kb > 0 || jj > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit_pair(&empty_bar[slot]);
          }
          __syncwarp();
          ++n; gpos += 3; if (gpos >= kPcNG) gpos -= kPcNG;
        }
        if (ok && leader) umma_commit_pair(&acc_full[1]);
        __syncwarp();
      }
    }
  } else if (run && warp >= 2 && warp < 10) {
    // ------------------------------------------------------------------ epilogues: one row, two 32-column chunks of one 64-column group per thread
    constexpr int kEpiThreads = 256;
    const int et = static_cast<int>(threadIdx.x) - 64;
    const int q = warp & 3, half = (warp - 2) >> 2;
    const int rloc = q * 32 + lane;
    const int m = row0 + rloc;                                   // kernel row
    const uint32_t trow = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    const int G = W / kStatCols;                                 // 64-column groups per row
    const int per = p.cfg ? 64 : 128;                            // tokens per row block
    const int own = per / kPcColTiles;                           // tokens this CTA updates
    const int tk_row = p.cfg ? (rloc & 63) : rloc;               // the row's token within the block
    bool ok = true;
    auto epi_sync = [&]() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory"); };
    // Waits are taken by one thread; the others learn the outcome after the barrier (uniform control flow).
    auto publish = [&](bool mine) { if (et == 0 && !mine) *epi_ok_s = 0; epi_sync(); ok = *epi_ok_s != 0; };
    auto meet_wait = [&](int idx) {      // every CTA of the group has passed meeting point idx
      bool w = true;
      if (et == 0 && ok) {
        w = pc_wait_count(ctr, static_cast<unsigned>(kPcGroup) * static_cast<unsigned>(idx + 1), p.err);
        if (w) pc_flag_set(meet_seen_s, static_cast<uint32_t>(idx + 1)); else ch_fail(p.err, DEV_ERR_EPI_WAIT, 8, idx);
      }
      publish(w);
    };
    auto meet_arrive = [&]() {           // after a barrier among the epilogue threads: their global writes are ordered before
      if (et == 0) pc_arrive(ctr);   // release: cumulative over the writes the barrier ordered before it
    };
    // The accumulators may be overwritten once every epilogue warp of the pair has read its part: each warp says so
    // right after its last read, before the arithmetic on what it read.
    auto release_acc = [&]() {
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(acc_empty), 0));
    };
    auto stage_act = [&](int c, const float* v) {
      uint8_t* row = stage_out + (c >> 1) * (kTileM * 128) + rloc * 128;
      ACT o[kChunk];
#pragma unroll
      for (int j = 0; j < kChunk; ++j) o[j] = to_act<ACT>(v[j]);
#pragma unroll
      for (int i = 0; i < 4; ++i)
        *reinterpret_cast<uint4*>(row + ((((c & 1) * 4 + i) ^ (rloc & 7)) << 4)) = reinterpret_cast<const uint4*>(o)[i];
    };
    // Update phase: x <- x_T (ft == 0) or the end of step ft (eps reduction over the column groups, guidance, Eq. 3)
    // for the tokens this CTA owns.
    auto update = [&](int ft) {
      const int tq = p.cfg ? (et >> 5) : (et >> 4), rep = p.cfg ? ((et >> 4) & 1) : 0, e = et & 15;
      const int i = tile_m * per + tile_n * own + tq;           // token
      if (ft == 0) {
        if (rep == 0 && i < p.R && e < p.C) {
          const float v = p.x_T[static_cast<size_t>(i) * p.C + e];
          p.x[static_cast<size_t>(i) * p.C + e] = v;
          if (p.traj_x) p.traj_x[static_cast<size_t>(i) * p.C + e] = v;
        }
        return;
      }
      {
        const int row = row0 + rep * 64 + tile_n * own + tq;
        const float* src = p.epart + (static_cast<size_t>(row) * G) * kCPad + e;
        float a[16];
#pragma unroll
        for (int g = 0; g < 16; ++g) a[g] = __ldcg(src + g * kCPad);      // G = 16 (W = 1024)
        float sum = 0.0f;
#pragma unroll
        for (int g = 0; g < 16; ++g) sum += a[g];
        eh[et] = sum + p.bout[e];
      }
      epi_sync();
      if (rep == 0 && i < p.R && e < p.C) {
        const size_t o = static_cast<size_t>(i) * p.C + e;
        float ee = eh[et];
        if (p.cfg) ee = cfg_combine(eh[et], eh[et + 16], p.cfg_scale);
        const float xo = __ldcg(p.x + o);
        const float mu = ddpm_mean(p.sched[ft - 1], xo, p.sched[T + ft - 1], ee);
        const float xn = ddpm_sample(mu, p.sched[2 * T + ft - 1], p.eps[static_cast<size_t>(ft - 1) * p.R * p.C + o]);
        if (!(fabsf(xn) <= 3.0e38f)) *p.status = 1;
        if (ft == 1) {
          p.mu1[o] = mu;
          if (p.x1) p.x1[o] = xo;
          if (p.sample_last && p.x0) p.x0[o] = xn;
        } else {
          p.x[o] = xn;
          if (p.traj_x) {
            const size_t slot = static_cast<size_t>(p.R) * p.C;
            p.traj_x[static_cast<size_t>(T - ft + 1) * slot + o] = xn;
            p.traj_mu[static_cast<size_t>(T - ft) * slot + o] = mu;
          }
        }
      }
    };
    int gp = 0, deps = 0;
    for (int si = 0; si < T && ok; ++si) {
      const int t = T - si;
      // ---- update (meeting point si NS)
      if (si > 0) meet_wait((si - 1) * NS + NS - 1);
      if (!ok) break;
      update(si == 0 ? 0 : t + 1);
      epi_sync();
      meet_arrive();
      for (int ph = 0; ph < NP && ok; ++ph, ++gp) {
        const bool dep = has_dep(ph);
        const bool is_w1 = dep && (ph & 1), is_gate = dep && !(ph & 1), is_f = ph == NP - 1, is_b = ph == 0;
        const bool last_gate = ph == 2 * L;
        float* bias_s = bias_all + (gp & 1) * 384;
        if (et < 128) {
          const float* const* bp = p.bias + ph * 3;
#pragma unroll
          for (int u = 0; u < 3; ++u) { const float* b = bp[u]; bias_s[u * 128 + et] = b ? b[n_base + et] : 0.0f; }
        }
        // the preceding phase's outputs of the whole group (x, LayerNorm partials, activations) are in place
        meet_wait(si * NS + ph);
        if (!ok) break;
        float mean = 0.0f, rstd = 0.0f;
        if (is_w1 || is_f) {
          // LayerNorm statistics of the row from its 16 partials.  The row block's partials (16 KB, contiguous) come in
          // with coalesced loads through the idle output buffer: row-per-thread loads (32 lines per instruction) held up
          // the SM's TMA traffic for about 3 k cycles.
          const float4* src = reinterpret_cast<const float4*>(p.stats) + static_cast<size_t>(row0) * (G / 2);
          float4* st4 = reinterpret_cast<float4*>(stage_out);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int idx = et + kEpiThreads * k, r = idx >> 3, j = idx & 7;
            st4[r * 8 + (j ^ (r & 7))] = __ldcg(src + idx);
          }
          epi_sync();
          float4 b[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) b[j] = st4[rloc * 8 + (j ^ (rloc & 7))];
          float sum = 0.0f, m2 = 0.0f, qq = 0.0f;
#pragma unroll
          for (int j = 0; j < 8; ++j) { sum += b[j].x; sum += b[j].z; m2 += b[j].y; m2 += b[j].w; }
          mean = sum / static_cast<float>(G);
#pragma unroll
          for (int j = 0; j < 8; ++j) { const float d0 = b[j].x - mean, d1 = b[j].z - mean; qq = fmaf(d0, d0, qq); qq = fmaf(d1, d1, qq); }
          rstd = 1.0f / sqrtf(fmaf(static_cast<float>(kStatCols), qq, m2) / static_cast<float>(W) + 1e-6f);
        }
        if (is_b) {
          for (int e = et; e < per * kCPad; e += kEpiThreads) {
            const int i = tile_m * per + (e >> 4), cc = e & 15;
            xg[e] = (i < p.R && cc < p.C) ? __ldcg(p.x + static_cast<size_t>(i) * p.C + cc) : 0.0f;
          }
          epi_sync();
        }
        {
          bool w = true;
          if (et == 0) {
            w = ch_wait<false>(&acc_full[0], gp & 1, p.err);
            if (w && dep) w = ch_wait<false>(&acc_full[1], deps & 1, p.err);
            if (!w) ch_fail(p.err, DEV_ERR_EPI_WAIT, 3, ph);
          }
          publish(w);
        }
        if (!ok) break;
        if (dep) ++deps;
        tc_fence_after_sync();
        // one code path per kind of phase (each keeps only its own accumulators in registers)
        if (is_w1) {
#pragma unroll
          for (int ci = 0; ci < 2; ++ci) {
            const int c = 2 * half + ci;                                  // 32-column chunk of the tile
            float a0[kChunk], a1[kChunk], am[kChunk];
            const uint32_t colp = kPcAccP + (c >> 1) * 128 + (c & 1) * kChunk;
            tmem_ld32(trow + colp, a0);                                   // P1
            tmem_ld32(trow + colp + kStatCols, a1);                       // P2
            tmem_ld32(trow + kPcAccM + c * kChunk, am);
            tmem_ld_wait();
            if (ci == 1) release_acc();
            const float* k0 = bias_s + c * kChunk;
            const float* k1 = bias_s + 128 + c * kChunk;
#pragma unroll
            for (int j = 0; j < kChunk; ++j) {
              const float t1 = __fsub_rn(am[j], __fmul_rn(mean, __fadd_rn(a0[j], k0[j])));
              am[j] = silu_t<true>(fmaf(rstd, t1, __fadd_rn(a1[j], k1[j])));
            }
            stage_act(c, am);
          }
        } else if (is_gate) {
          RowState rs;
          rs.pm = 0.0f; rs.pm2 = 0.0f; rs.pn = 0.0f;
#pragma unroll
          for (int ci = 0; ci < 2; ++ci) {
            const int c = 2 * half + ci;
            float a0[kChunk], a1[kChunk], am[kChunk], hv[kChunk];
            const uint32_t colp = kPcAccP + (last_gate ? c * kChunk : (c >> 1) * 128 + (c & 1) * kChunk);
            tmem_ld32(trow + colp, a0);                                   // gate
            if (!last_gate) tmem_ld32(trow + colp + kStatCols, a1);       // next block's scale
            tmem_ld32(trow + kPcAccM + c * kChunk, am);
            tmem_ld32(trow + kPcAccH + c * kChunk, hv);
            tmem_ld_wait();
            if (ci == 1) release_acc();
            gate_res_chunk(a0, am, bias_s + c * kChunk, bias_s + 128 + c * kChunk, hv, rs);
            tmem_st32(trow + kPcAccH + c * kChunk, hv);
            if (!last_gate) {
              const float* k2 = bias_s + 256 + c * kChunk;
#pragma unroll
              for (int j = 0; j < kChunk; ++j) hv[j] = __fmul_rn(hv[j], __fadd_rn(1.0f, __fadd_rn(a1[j], k2[j])));
              stage_act(c, hv);
            }
          }
          tmem_st_wait();
          reinterpret_cast<float2*>(p.stats)[static_cast<size_t>(m) * G + tile_n * 2 + half] = make_float2(rs.pm, rs.pm2);
        } else if (is_f) {
          float eacc[kCPad];
#pragma unroll
          for (int e = 0; e < kCPad; ++e) eacc[e] = 0.0f;
#pragma unroll
          for (int ci = 0; ci < 2; ++ci) {
            const int c = 2 * half + ci;
            float a0[kChunk], a1[kChunk], hv[kChunk];
            const uint32_t colp = kPcAccP + (c >> 1) * 128 + (c & 1) * kChunk;
            tmem_ld32(trow + colp, a0);                                   // shift
            tmem_ld32(trow + colp + kStatCols, a1);                       // scale
            tmem_ld32(trow + kPcAccH + c * kChunk, hv);
            tmem_ld_wait();
            if (ci == 1) release_acc();
            const float* k0 = bias_s + c * kChunk;
            const float* k1 = bias_s + 128 + c * kChunk;
            const float* wc = wout_s + c * kChunk * kCPad;
#pragma unroll
            for (int j = 0; j < kChunk; ++j) {
              const float uf = fmaf(__fmul_rn(__fsub_rn(hv[j], mean), rstd), __fadd_rn(1.0f, a1[j] + k1[j]), a0[j] + k0[j]);
              const float4* w4 = reinterpret_cast<const float4*>(wc + j * kCPad);
#pragma unroll
              for (int c4 = 0; c4 < kCPad / 4; ++c4) {
                const float4 w = w4[c4];
                eacc[4 * c4 + 0] = fmaf(uf, w.x, eacc[4 * c4 + 0]); eacc[4 * c4 + 1] = fmaf(uf, w.y, eacc[4 * c4 + 1]);
                eacc[4 * c4 + 2] = fmaf(uf, w.z, eacc[4 * c4 + 2]); eacc[4 * c4 + 3] = fmaf(uf, w.w, eacc[4 * c4 + 3]);
              }
            }
          }
          float4* d = reinterpret_cast<float4*>(p.epart + (static_cast<size_t>(m) * G + tile_n * 2 + half) * kCPad);
#pragma unroll
          for (int c4 = 0; c4 < kCPad / 4; ++c4) d[c4] = make_float4(eacc[4 * c4], eacc[4 * c4 + 1], eacc[4 * c4 + 2], eacc[4 * c4 + 3]);
        } else {
          // boundary: h = Win x + bin for this row and the tile's columns; a' = h (1 + scale_0)
          float xr[kCPad];
          {
            const float4* xq = reinterpret_cast<const float4*>(xg + tk_row * kCPad);
#pragma unroll
            for (int c4 = 0; c4 < kCPad / 4; ++c4) { const float4 v = xq[c4]; xr[4 * c4] = v.x; xr[4 * c4 + 1] = v.y; xr[4 * c4 + 2] = v.z; xr[4 * c4 + 3] = v.w; }
          }
          float pm = 0.0f, pm2 = 0.0f;
#pragma unroll
          for (int ci = 0; ci < 2; ++ci) {
            const int c = 2 * half + ci;
            float a1[kChunk], hv[kChunk];
            tmem_ld32(trow + kPcAccP + (c >> 1) * 128 + (c & 1) * kChunk + kStatCols, a1);   // scale of block 0
            if (ci == 1) { tmem_ld_wait(); release_acc(); }
            float sum = 0.0f;
#pragma unroll
            for (int j0 = 0; j0 < kChunk; j0 += 4) {          // four independent chains
              float acc4[4];
#pragma unroll
              for (int u = 0; u < 4; ++u) acc4[u] = bin_s[c * kChunk + j0 + u];
#pragma unroll
              for (int c4 = 0; c4 < kCPad / 4; ++c4) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                  const float4 w = reinterpret_cast<const float4*>(win_s + (c * kChunk + j0 + u) * kCPad)[c4];
                  acc4[u] = fmaf(w.x, xr[4 * c4], acc4[u]); acc4[u] = fmaf(w.y, xr[4 * c4 + 1], acc4[u]);
                  acc4[u] = fmaf(w.z, xr[4 * c4 + 2], acc4[u]); acc4[u] = fmaf(w.w, xr[4 * c4 + 3], acc4[u]);
                }
              }
#pragma unroll
              for (int u = 0; u < 4; ++u) { hv[j0 + u] = acc4[u]; sum += acc4[u]; }
            }
            const float mu = sum * (1.0f / kChunk);
            float m2 = 0.0f;
#pragma unroll
            for (int j = 0; j < kChunk; ++j) { const float dd = hv[j] - mu; m2 = fmaf(dd, dd, m2); }
            if (ci == 0) { pm = mu; pm2 = m2; } else chan_merge_equal(pm, pm2, mu, m2, static_cast<float>(kChunk));
            tmem_st32(trow + kPcAccH + c * kChunk, hv);
            tmem_ld_wait();
            const float* k0 = bias_s + c * kChunk;
#pragma unroll
            for (int j = 0; j < kChunk; ++j) hv[j] = __fmul_rn(hv[j], __fadd_rn(1.0f, __fadd_rn(a1[j], k0[j])));
            stage_act(c, hv);
          }
          tmem_st_wait();
          reinterpret_cast<float2*>(p.stats)[static_cast<size_t>(m) * G + tile_n * 2 + half] = make_float2(pm, pm2);
        }
        const bool stores = is_w1 || is_b || (is_gate && !last_gate);
        if (stores) fence_proxy_async_smem();
        tc_fence_before_sync();   // orders the TMEM reads before the barrier that releases the accumulators
        epi_sync();
        if (et == 0) {
          if (stores) {
            const CUtensorMap* tmo = is_w1 ? &tmV : &tmAp;
            tma_store_2d(tmo, stage_out, n_base, row0);
            tma_store_2d(tmo, stage_out + kTileM * 128, n_base + 64, row0);
            tma_store_commit();
            tma_store_wait_all();   // complete before the release below; the readers fence before their TMA loads
          }
        }
        meet_arrive();
      }
    }
    // ---- the last step's update
    if (ok) meet_wait((T - 1) * NS + NS - 1);
    if (ok) update(1);
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive(); cluster_wait();   // neither CTA leaves while the pair's MMAs or signals may touch it
  if (warp == 1) tmem_dealloc_pair(tmem_base, 512);
}

// s_t = SiLU(cz + te_t) of every step, in the kernel's row order and operand format: s_all[(t - 1) rows + rho][col];
// rows of tokens beyond R are zero.
template <typename ACT>
__global__ void __launch_bounds__(128) pc_cond_all_kernel(const float* __restrict__ cz, const float* __restrict__ te,
                                                          ACT* __restrict__ s_all, int R, int cfg, int W, int rows) {
  const int t = blockIdx.y, rho = blockIdx.x;
  int rep;
  const int i = pc_row_token(rho, cfg, &rep);
  uint4* dst = reinterpret_cast<uint4*>(s_all + (static_cast<size_t>(t) * rows + rho) * W);     // 8 values per store
  if (i >= R) {
    for (int j = threadIdx.x; j < W / 8; j += blockDim.x) dst[j] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const float4* c4 = reinterpret_cast<const float4*>(cz + (static_cast<size_t>(rep) * R + i) * W);
  const float4* t4 = reinterpret_cast<const float4*>(te + static_cast<size_t>(t) * W);
  for (int j = threadIdx.x; j < W / 8; j += blockDim.x) {
    const float4 a = c4[2 * j], b = c4[2 * j + 1], ta = __ldg(t4 + 2 * j), tb = __ldg(t4 + 2 * j + 1);
    __align__(16) ACT o[8];
    o[0] = to_act<ACT>(silu_f(a.x + ta.x)); o[1] = to_act<ACT>(silu_f(a.y + ta.y));
    o[2] = to_act<ACT>(silu_f(a.z + ta.z)); o[3] = to_act<ACT>(silu_f(a.w + ta.w));
    o[4] = to_act<ACT>(silu_f(b.x + tb.x)); o[5] = to_act<ACT>(silu_f(b.y + tb.y));
    o[6] = to_act<ACT>(silu_f(b.z + tb.z)); o[7] = to_act<ACT>(silu_f(b.w + tb.w));
    dst[j] = *reinterpret_cast<const uint4*>(o);
  }
}

}  // namespace csd
