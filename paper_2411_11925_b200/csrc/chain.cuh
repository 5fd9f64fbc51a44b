// One kernel for a whole denoising chain (all T steps of Eq. 3 for one head): the launch-bound regime.
//
// A head is a per-token MLP, so a block of 128 rows never needs another block's data.  One thread-block
// cluster owns one row block for the whole chain; its W/128 CTAs each own a 128-column slice of every
// layer's output.  Between layers the slices meet through global memory (L2): a CTA writes its slice of
// the activation, signals every CTA of the cluster (remote add to a counter in its shared memory), and the next layer's TMA
// loads start once all slices are signalled.  No kernel boundary, no grid-wide dependency: a row block
// runs ahead of the others freely.
//
// Per CTA: the fp32 residual stream h (its 128 x 128 slice) lives in shared memory for the whole chain; a
// 4-slot TMA ring feeds tcgen05 MMAs into three TMEM accumulators (AdaLN shift|scale 256 columns, gate
// 128, MLP 128), so the products that depend only on the condition vector s (modulation of the next
// block, gate of this block) are issued while this block's dependent layers are in their epilogues.
// Warp 0 requests activation tiles, the last warp weight tiles (one thread sustains about one TMA request
// per 300 clk), warp 1 issues MMAs, 16 epilogue warps (one row x 32 columns per thread).  The activations
// u, v, s are kept in the kernel's own row order (row block after row block), so a tile is one TMA box even
// with guidance, where a row block holds 64 conditional rows and their 64 unconditional twins.
//
// The arithmetic (accumulation order, epilogue formulas, LayerNorm and eps_hat partial layout) is that of
// the layer-by-layer kernels; the two paths give the same bits.
#pragma once
#include "gemm.cuh"
#include "rowops.cuh"

namespace csd {

constexpr int kChSlots = 4;                     // ring slots: [A tile 16 KB | B tile 16 KB]
constexpr int kChSlotBytes = 32768;
constexpr int kChEpiWarps = 16;
constexpr int kChEpiThreads = kChEpiWarps * 32;
constexpr int kChThreads = kChEpiThreads + 96;   // + TMA (activations), MMA, TMA (weights)
constexpr int kChHBytes = kTileM * kTileN * 4;  // h slice: 4 chunks of [128 rows][128 B], 128-byte swizzle
constexpr int kChWoutBytes = kTileN * kCPad * 4;
constexpr int kChXBytes = kTileM * kCPad * 4;   // x of the row block's tokens
constexpr int kChXchBytes = kTileM * kCPad * 4; // exchange between column-chunk pairs
constexpr int kChBiasBytes = 2 * 256 * 4;       // two buffers of two 128-column bias slices
constexpr int kChSmemBytes = 1024 + kChSlots * kChSlotBytes + kChHBytes + kChWoutBytes + kChXBytes + kChXchBytes +
                             kChBiasBytes + 256;
constexpr uint32_t kAccMod = 0, kAccGate = 256, kAccMain = 384;   // TMEM columns of the three accumulators
constexpr int kChMaxCluster = 8;                // portable cluster size: W <= 1024

enum ChainAcc : int { ACC_MOD = 0, ACC_GATE = 1, ACC_MAIN = 2 };

struct ChainParams {
  const CUtensorMap* wmaps;   // device: per block Wss (256-row boxes), Wg, W1, W2 (128-row boxes); then Wfss
  const CUtensorMap* amaps;   // device: s for even t, s for odd t, u, v (boxes of 128 rows x 64 columns)
  int R, cfg, W, L, T, C, sample_last;
  float cfg_scale;
  const float* sched;         // device [3 T]: a, b, sigma
  const float* cz;            // [Rh, W]
  const float* te;            // [T, W]
  const float* const* bias;   // device [5 L + 2]: per block shift, scale, b1, gate, b2 biases; final shift, scale
  const float *win, *bin, *wout_t, *bout;
  void* s[2];                 // s of even / odd t, [row blocks * 128, W], the kernel's row order
  void *u, *v;                // same shape and order
  float* stats;               // [Rh, W/64, 2]
  float* epart;               // [Rh, W/64, 16]
  const float *x_T, *eps;     // [R, C], [T, R, C]
  float *x0, *mu1, *x1;       // outputs of the last step (x0, x1 may be null)
  int* err;
};

// Bounded wait that also gives up once any kernel of the context has raised the error flag.
template <bool CLUSTER>
__device__ __forceinline__ bool ch_wait(uint64_t* bar, uint32_t parity, const int* err) {
  long long t0 = 0;
  uint32_t spins = 0;
  for (;;) {
    if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
    if ((++spins & 1023u) == 0u) {
      if (*reinterpret_cast<const volatile int*>(err) != 0) return false;
      const long long now = clock64();
      if (t0 == 0) t0 = now;
      else if (now - t0 > 4000000000ll) return false;
    }
  }
}

// Waits until the cluster-wide phase counter has reached `target` (bounded like ch_wait).  A counter, not an
// mbarrier: a waiter may find several phases completed since it last looked, which a phase parity cannot tell.
__device__ __forceinline__ bool ch_wait_count(const uint32_t* cnt, uint32_t target, const int* err) {
  long long t0 = 0;
  uint32_t spins = 0;
  for (;;) {
    if (ld_acquire_cluster(cnt) >= target) return true;
    if ((++spins & 1023u) == 0u) {
      if (*reinterpret_cast<const volatile int*>(err) != 0) return false;
      const long long now = clock64();
      if (t0 == 0) t0 = now;
      else if (now - t0 > 4000000000ll) return false;
    }
  }
}

// 19 warps: the register file is split over four schedulers, so five warps on one of them cap a thread at
// 96 registers.
// First failing wait of a chain kernel: role (DevErr) | site << 4 | (count & 0xffff) << 8 | (block & 0x7f) << 24.
__device__ __forceinline__ void ch_fail(int* err, int role, int site, int count) {
  atomicCAS(err, 0, role | (site << 4) | ((count & 0xffff) << 8) | ((static_cast<int>(blockIdx.x) & 0x7f) << 24));
}

template <typename ACT, int AB_FMT>
__global__ void __launch_bounds__(kChThreads, 1) chain_kernel(const ChainParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* ring = smem;
  uint8_t* h_s = ring + kChSlots * kChSlotBytes;
  float* wout_s = reinterpret_cast<float*>(h_s + kChHBytes);
  float* x_s = wout_s + kChWoutBytes / 4;     // [tokens of the block][16]
  float* xch_s = x_s + kChXBytes / 4;         // [128 rows][16]
  float* bias_s = xch_s + kChXchBytes / 4;    // [2][256]
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(bias_s + 512);
  uint64_t* empty_bar = full_bar + kChSlots;
  uint64_t* acc_full = empty_bar + kChSlots;  // [3]
  uint64_t* acc_empty = acc_full + 3;         // [3]
  uint32_t* sync_cnt = reinterpret_cast<uint32_t*>(acc_empty + 3);   // phases signalled by the cluster's CTAs, nc per phase
  uint32_t* tmem_base_s = sync_cnt + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int W = p.W, L = p.L, T = p.T;
  const int nc = W / kTileN;                                 // CTAs per cluster
  const int j = static_cast<int>(cluster_ctarank());         // this CTA's column slice
  const int tb = static_cast<int>(blockIdx.x) / nc;          // token block of the cluster
  const int TB = p.cfg ? kTileM / 2 : kTileM;                // tokens per block (guidance: 64 cond + 64 uncond rows)
  const int nrep = p.cfg ? 2 : 1;
  const int nkb = W / kBlockK;
  const int G = W / kStatCols;
  const int n_base = j * kTileN;
  const int row0 = tb * kTileM;   // first row of the block in u, v, s
  const int syncs_per_step = 3 * L + 2;

  const bool run = *reinterpret_cast<const volatile int*>(p.err) == 0;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kChSlots; ++s) { mbar_init(&full_bar[s], 2); mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < 3; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 1); }
    *sync_cnt = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(tmem_base_s, 512); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive(); cluster_wait();        // every CTA's barriers exist before anything signals them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_base_s;

  if (run && warp == 0) {
    // ------------------------------------------------------------------ TMA requests
    const bool leader = elect_one();
    bool ok = true;
    int it = 0;
    auto sync_until = [&](int idx) {   // phase idx has been signalled by every CTA of the cluster
      if (ok) { ok = ch_wait_count(sync_cnt, static_cast<uint32_t>((idx + 1) * nc), p.err); if (!ok && leader) ch_fail(p.err, DEV_ERR_TMA_WAIT, 1, idx); }
      fence_proxy_async_all();
    };
    auto slot_free = [&](int c) {   // slot of ring counter c is free again
      if (ok && c >= kChSlots) { ok = ch_wait<false>(&empty_bar[c % kChSlots], ((c / kChSlots) & 1) ^ 1, p.err); if (!ok && leader) ch_fail(p.err, DEV_ERR_TMA_WAIT, 2, c); }
    };
    // N = 128 segment: one slot per k-block
    auto seg128 = [&](const CUtensorMap* ta) {
      for (int kb = 0; kb < nkb && ok; ++kb, ++it) {
        slot_free(it);
        if (ok && leader) {
          const int s = it % kChSlots;
          uint8_t* dst = ring + s * kChSlotBytes;
          mbar_arrive_expect_tx(&full_bar[s], 16384);
          tma_load_2d(dst, ta, &full_bar[s], kb * kBlockK, row0);
        }
        __syncwarp();
      }
    };
    // N = 256 segment (packed shift|scale rows): two slots per k-block, the 32 KB weight tile runs from
    // the second half of the first slot through the first half of the second
    auto seg256 = [&](const CUtensorMap* ta) {
      for (int kb = 0; kb < nkb && ok; ++kb, it += 2) {
        slot_free(it); slot_free(it + 1);
        if (ok && leader) {
          const int s = it % kChSlots;
          uint8_t* dst = ring + s * kChSlotBytes;
          mbar_arrive_expect_tx(&full_bar[s], 16384);
          tma_load_2d(dst, ta, &full_bar[s], kb * kBlockK, row0);
          mbar_arrive(&full_bar[s + 1]);
        }
        __syncwarp();
      }
    };
    const CUtensorMap* tm_u = p.amaps + 2;
    const CUtensorMap* tm_v = p.amaps + 3;
    sync_until(0);
    seg256(p.amaps + (T & 1));                                        // modulation of block 0, step T
    for (int si = 0; si < T && ok; ++si) {
      const int t = T - si, base = 1 + si * syncs_per_step;
      const CUtensorMap* tm_s = p.amaps + (t & 1);
      for (int k = 0; k < L && ok; ++k) {
        sync_until(base + 3 * k);       seg128(tm_u);                  // u W1^T
        seg128(tm_s);                                                 // s Wg^T
        sync_until(base + 3 * k + 1);   seg128(tm_v);                  // v W2^T
        seg256(tm_s);                                                 // modulation of block k + 1 / final
      }
      if (t > 1) seg256(p.amaps + ((t - 1) & 1));                     // modulation of block 0, next step
    }
    if (!ok && leader) ch_fail(p.err, DEV_ERR_TMA_WAIT, 0, 0);
    __syncwarp();
  } else if (run && warp == kChEpiWarps + 2) {
    // ------------------------------------------------------------------ TMA requests, weight tiles
    // (never wait for the cluster: the ring fills with the weights of layers whose activations are not ready yet)
    const bool leader = elect_one();
    bool ok = true;
    int it = 0;
    auto slot_free = [&](int c) {
      if (ok && c >= kChSlots) { ok = ch_wait<false>(&empty_bar[c % kChSlots], ((c / kChSlots) & 1) ^ 1, p.err); if (!ok && leader) ch_fail(p.err, DEV_ERR_TMA_WAIT, 8, c); }
    };
    auto seg128 = [&](const CUtensorMap* tw) {
      for (int kb = 0; kb < nkb && ok; ++kb, ++it) {
        slot_free(it);
        if (ok && leader) {
          const int s = it % kChSlots;
          mbar_arrive_expect_tx(&full_bar[s], 16384);
          tma_load_2d(ring + s * kChSlotBytes + 16384, tw, &full_bar[s], kb * kBlockK, n_base);
        }
        __syncwarp();
      }
    };
    auto seg256 = [&](const CUtensorMap* tw) {
      for (int kb = 0; kb < nkb && ok; ++kb, it += 2) {
        slot_free(it); slot_free(it + 1);
        if (ok && leader) {
          const int s = it % kChSlots;
          mbar_arrive_expect_tx(&full_bar[s], 32768);
          tma_load_2d(ring + s * kChSlotBytes + 16384, tw, &full_bar[s], kb * kBlockK, 2 * n_base);
          mbar_arrive(&full_bar[s + 1]);
        }
        __syncwarp();
      }
    };
    seg256(p.wmaps);
    for (int si = 0; si < T && ok; ++si) {
      for (int k = 0; k < L && ok; ++k) {
        const CUtensorMap* wk = p.wmaps + 4 * k;
        seg128(wk + 2); seg128(wk + 1); seg128(wk + 3); seg256(wk + 4);
      }
      if (si + 1 < T) seg256(p.wmaps);
    }
    __syncwarp();
  } else if (run && warp == 1) {
    // ------------------------------------------------------------------ MMA issue
    const bool leader = elect_one();
    constexpr uint32_t idesc128 = umma_idesc_f16(128, AB_FMT), idesc256 = umma_idesc_f16(256, AB_FMT);
    bool ok = true;
    int it = 0;
    int n_use[3] = {0, 0, 0};
    auto acc_begin = [&](int a) {   // the epilogue has drained the accumulator's previous contents
      if (ok && n_use[a] >= 1) { ok = ch_wait<false>(&acc_empty[a], (n_use[a] - 1) & 1, p.err); if (!ok && leader) ch_fail(p.err, DEV_ERR_MMA_WAIT, 3 + a, n_use[a]); }
      ++n_use[a];
      tc_fence_after_sync();
    };
    auto seg128 = [&](int a, uint32_t col) {
      acc_begin(a);
      for (int kb = 0; kb < nkb && ok; ++kb, ++it) {
        const int s = it % kChSlots;
        ok = ch_wait<false>(&full_bar[s], (it / kChSlots) & 1, p.err);
        if (!ok) { if (leader) ch_fail(p.err, DEV_ERR_MMA_WAIT, 6, it); break; }
        tc_fence_after_sync();
        if (leader) {
          const uint32_t sa = smem_u32(ring + s * kChSlotBytes);
          const uint64_t da = umma_smem_desc_sw128(sa), db = umma_smem_desc_sw128(sa + 16384);
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k) umma_f16(tmem_base + col, da + 2 * k, db + 2 * k, idesc128, (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit(&empty_bar[s]);
        }
        __syncwarp();
      }
      if (ok && leader) umma_commit(&acc_full[a]);
      __syncwarp();
    };
    auto seg256 = [&](int a, uint32_t col) {
      acc_begin(a);
      for (int kb = 0; kb < nkb && ok; ++kb, it += 2) {
        const int s = it % kChSlots;
        ok = ch_wait<false>(&full_bar[s], (it / kChSlots) & 1, p.err);
        if (ok) ok = ch_wait<false>(&full_bar[s + 1], ((it + 1) / kChSlots) & 1, p.err);
        if (!ok) { if (leader) ch_fail(p.err, DEV_ERR_MMA_WAIT, 7, it); break; }
        tc_fence_after_sync();
        if (leader) {
          const uint32_t sa = smem_u32(ring + s * kChSlotBytes);
          const uint64_t da = umma_smem_desc_sw128(sa), db = umma_smem_desc_sw128(sa + 16384);
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k) umma_f16(tmem_base + col, da + 2 * k, db + 2 * k, idesc256, (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit(&empty_bar[s]);
          umma_commit(&empty_bar[s + 1]);
        }
        __syncwarp();
      }
      if (ok && leader) umma_commit(&acc_full[a]);
      __syncwarp();
    };
    seg256(ACC_MOD, kAccMod);
    for (int si = 0; si < T && ok; ++si) {
      for (int k = 0; k < L && ok; ++k) {
        seg128(ACC_MAIN, kAccMain);
        seg128(ACC_GATE, kAccGate);
        seg128(ACC_MAIN, kAccMain);
        seg256(ACC_MOD, kAccMod);
      }
      if (si + 1 < T) seg256(ACC_MOD, kAccMod);
    }
    if (!ok && leader) ch_fail(p.err, DEV_ERR_MMA_WAIT, 0, 0);
    __syncwarp();
  } else if (run && warp >= 2 && warp < kChEpiWarps + 2) {
    // ------------------------------------------------------------------ epilogues
    const int et = static_cast<int>(threadIdx.x) - 64;
    const int ew = warp - 2;
    const int q = warp & 3, cg = ew >> 2;          // TMEM lane quarter, 32-column chunk of the slice
    const int rloc = q * 32 + lane;
    const int rep = p.cfg ? (rloc >> 6) : 0;
    const int token = tb * TB + (p.cfg ? (rloc & 63) : rloc);
    const bool valid = token < p.R;
    const int m = token + rep * p.R;               // row of the caller's layout
    const int n0 = n_base + cg * kChunk;
    const uint32_t trow = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    uint8_t* h_chunk = h_s + cg * (kTileM * 128);
    const size_t mi = static_cast<size_t>(row0 + rloc);   // row in u, v, s
    ACT* u_out = reinterpret_cast<ACT*>(p.u);
    ACT* v_out = reinterpret_cast<ACT*>(p.v);
    bool ok = true;
    int n_full[3] = {0, 0, 0}, bias_buf = 0;
    float next_bias = 0.0f;

    auto sync_until = [&](int idx) {
      int w = 1;
      if (ok && lane == 0) { w = ch_wait_count(sync_cnt, static_cast<uint32_t>((idx + 1) * nc), p.err) ? 1 : 0; if (!w) ch_fail(p.err, DEV_ERR_EPI_WAIT, 1, idx); }
      w = __shfl_sync(0xffffffffu, w, 0);
      if (!w) ok = false;
    };
    auto acc_wait = [&](int a) {
      int w = 1;
      if (ok && lane == 0) { w = ch_wait<false>(&acc_full[a], n_full[a] & 1, p.err) ? 1 : 0; if (!w) ch_fail(p.err, DEV_ERR_EPI_WAIT, 3 + a, n_full[a]); }
      w = __shfl_sync(0xffffffffu, w, 0);
      if (!w) ok = false;
      ++n_full[a];
      tc_fence_after_sync();
    };
    // bias vectors of the phases, in the order the epilogues run: per block (shift, scale), (b1), (gate, b2); then
    // the final (shift, scale).  Thread et < 256 fetches element et % 128 of vector et / 128.
    auto bias_fetch = [&](int phase) {   // phase in [0, 3 L]
      if (et < 256) {
        const int k = phase / 3, r = phase % 3, v = et >> 7;
        const float* src = nullptr;
        if (phase == 3 * L) src = p.bias[5 * L + v];
        else if (r == 0) src = p.bias[5 * k + v];
        else if (r == 1) src = v == 0 ? p.bias[5 * k + 2] : nullptr;
        else src = p.bias[5 * k + 3 + v];
        next_bias = src ? src[n_base + (et & 127)] : 0.0f;
      }
    };
    // End of a phase: this CTA's stores are ordered before the signal that lets the cluster's TMA loads
    // read them; `release_mask` = accumulators this phase has drained.
    auto phase_end = [&](int release_mask) {
      if (et < 256) bias_s[(bias_buf ^ 1) * 256 + et] = next_bias;
      bias_buf ^= 1;
      tc_fence_before_sync();
      fence_proxy_async_all();
      asm volatile("bar.sync 1, %0;" ::"n"(kChEpiThreads) : "memory");
      if (et == 0 && ok) {
        for (int a = 0; a < 3; ++a)
          if (release_mask & (1 << a)) mbar_arrive(&acc_empty[a]);
        // one fence for the whole CTA's stores (ordered before it by the barrier), then relaxed signals
        __threadfence();
        const uint32_t sb = smem_u32(sync_cnt);
        for (int r = 0; r < nc; ++r) red_add_cluster(mapa_shared(sb, static_cast<uint32_t>(r)), 1u);
      }
    };
    // h = Win x + bin for this CTA's slice, its LayerNorm partials, from x_s
    auto input_proj = [&]() {
      const int g = ew & 1;                       // 64-column group of the slice
      const int na = n_base + g * kStatCols + lane, nb = na + 32;
      float wa[kCPad], wb[kCPad];
#pragma unroll
      for (int c4 = 0; c4 < kCPad / 4; ++c4) {
        const float4 qa = reinterpret_cast<const float4*>(p.win + static_cast<size_t>(na) * kCPad)[c4];
        const float4 qb = reinterpret_cast<const float4*>(p.win + static_cast<size_t>(nb) * kCPad)[c4];
        wa[4 * c4] = qa.x; wa[4 * c4 + 1] = qa.y; wa[4 * c4 + 2] = qa.z; wa[4 * c4 + 3] = qa.w;
        wb[4 * c4] = qb.x; wb[4 * c4 + 1] = qb.y; wb[4 * c4 + 2] = qb.z; wb[4 * c4 + 3] = qb.w;
      }
      const float ba = p.bin[na], bb = p.bin[nb];
      for (int ti = ew >> 1; ti < TB; ti += kChEpiWarps / 2) {
        float acc[2], mean, m2;
        input_proj_group(wa, wb, ba, bb, x_s + ti * kCPad, acc, mean, m2);
        const int tok = tb * TB + ti;
        for (int rp = 0; rp < nrep; ++rp) {
          const int l = rp * 64 + ti;             // local row (rp = 1 only with guidance, where ti < 64)
#pragma unroll
          for (int jj = 0; jj < 2; ++jj) {
            uint8_t* row = h_s + (g * 2 + jj) * (kTileM * 128) + l * 128;
            *reinterpret_cast<float*>(row + (((lane >> 2) ^ (l & 7)) << 4) + (lane & 3) * 4) = acc[jj];
          }
          if (lane == 0 && tok < p.R)
            reinterpret_cast<float2*>(p.stats)[static_cast<size_t>(tok + rp * p.R) * G + (n_base / kStatCols) + g] =
                make_float2(mean, m2);
        }
      }
    };
    // s(t') = SiLU(cz + te_{t'}) for this CTA's slice
    auto cond_vector = [&](int tp) {
      const int l = et >> 2, cc = et & 3;
      const int rp = p.cfg ? (l >> 6) : 0;
      const int tok = tb * TB + (p.cfg ? (l & 63) : l);
      if (tok < p.R) {
        const size_t off = static_cast<size_t>(tok + rp * p.R) * W + n_base + cc * kChunk;
        float a[kChunk], b[kChunk];
        load_chunk_f32(p.cz + off, a);
        load_chunk_f32(p.te + static_cast<size_t>(tp - 1) * W + n_base + cc * kChunk, b);
#pragma unroll
        for (int i = 0; i < kChunk; ++i) a[i] = silu_f(a[i] + b[i]);
        store_chunk<ACT>(reinterpret_cast<ACT*>(p.s[tp & 1]) + static_cast<size_t>(row0 + l) * W + n_base + cc * kChunk, a);
      }
    };

    // ---- chain prologue: x_T, h of step T, s of steps T and T - 1, constants
    for (int i = et; i < kTileN * kCPad; i += kChEpiThreads) wout_s[i] = p.wout_t[static_cast<size_t>(n_base) * kCPad + i];
    for (int i = et; i < TB * kCPad; i += kChEpiThreads) {
      const int tok = tb * TB + (i >> 4), c = i & 15;
      x_s[i] = (tok < p.R && c < p.C) ? p.x_T[static_cast<size_t>(tok) * p.C + c] : 0.0f;
    }
    bias_fetch(0);
    asm volatile("bar.sync 1, %0;" ::"n"(kChEpiThreads) : "memory");
    input_proj();
    cond_vector(T);
    if (T >= 2) cond_vector(T - 1);
    phase_end(0);                                                        // sync 0

    for (int si = 0; si < T; ++si) {
      const int t = T - si, base = 1 + si * syncs_per_step;
      for (int k = 0; k <= L; ++k) {
        // ---- AdaLN modulate of block k (k < L): u = LN(h)(1 + scale) + shift; k = L: final layer, eps_hat partials
        const bool fin = k == L;
        bias_fetch(fin ? 0 : 3 * k + 1);
        sync_until(base + 3 * k - 1);
        RowState rs;
        rs.mean = 0.0f; rs.rstd = 0.0f;
        if (ok && valid) row_stats<true>(p.stats, m, W, rs.mean, rs.rstd);
        acc_wait(ACC_MOD);
        if (ok) {
          float a0[kChunk], a1[kChunk], hv[kChunk];
          const uint32_t col0 = kAccMod + (cg >> 1) * 128 + (cg & 1) * kChunk;
          tmem_ld32(trow + col0, a0);
          tmem_ld32(trow + col0 + kStatCols, a1);
          load_swizzled_row32(h_chunk, rloc, hv);
          tmem_ld_wait();
          const float* b = bias_s + bias_buf * 256 + cg * kChunk;
          modulate_chunk(a0, a1, b, b + 128, hv, rs);
          if (!fin) {
            if (valid) store_chunk<ACT>(u_out + mi * W + n0, a0);
          } else {
#pragma unroll
            for (int c = 0; c < kCPad; ++c) rs.eacc[c] = 0.0f;
            outproj_chunk(a0, wout_s + cg * kChunk * kCPad, rs);
          }
        }
        if (fin) {
          // one eps_hat partial per row and 64-column group: (even chunk's sum) + (odd chunk's sum)
          for (int round = 0; round < 2; ++round) {
            if (cg == 2 * round + 1) {
#pragma unroll
              for (int c = 0; c < kCPad; ++c) xch_s[rloc * kCPad + c] = rs.eacc[c];
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kChEpiThreads) : "memory");
            if (cg == 2 * round && ok && valid) {
              float4* d = reinterpret_cast<float4*>(p.epart + (static_cast<size_t>(m) * G + (n_base / kStatCols) + round) * kCPad);
#pragma unroll
              for (int c4 = 0; c4 < kCPad / 4; ++c4)
                d[c4] = make_float4(rs.eacc[4 * c4] + xch_s[rloc * kCPad + 4 * c4], rs.eacc[4 * c4 + 1] + xch_s[rloc * kCPad + 4 * c4 + 1],
                                    rs.eacc[4 * c4 + 2] + xch_s[rloc * kCPad + 4 * c4 + 2], rs.eacc[4 * c4 + 3] + xch_s[rloc * kCPad + 4 * c4 + 3]);
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kChEpiThreads) : "memory");
          }
        }
        phase_end(1 << ACC_MOD);                                         // sync base + 3 k
        if (fin) break;

        // ---- first MLP layer: v = SiLU(u W1^T + b1)
        bias_fetch(3 * k + 2);
        acc_wait(ACC_MAIN);
        if (ok) {
          float a0[kChunk];
          tmem_ld32(trow + kAccMain + cg * kChunk, a0);
          tmem_ld_wait();
          const float* b = bias_s + bias_buf * 256 + cg * kChunk;
#pragma unroll
          for (int i = 0; i < kChunk; ++i) a0[i] = silu_t<true>(a0[i] + b[i]);
          if (valid) store_chunk<ACT>(v_out + mi * W + n0, a0);
        }
        phase_end(1 << ACC_MAIN);                                        // sync base + 3 k + 1

        // ---- second MLP layer, gate, residual: h += (s Wg^T + bg) (v W2^T + b2); LayerNorm partials
        bias_fetch(3 * k + 3);
        acc_wait(ACC_GATE);
        acc_wait(ACC_MAIN);
        RowState rg;
        rg.pm = 0.0f; rg.pm2 = 0.0f; rg.pn = 0.0f;
        if (ok) {
          float a0[kChunk], a1[kChunk], hv[kChunk];
          tmem_ld32(trow + kAccGate + cg * kChunk, a0);
          tmem_ld32(trow + kAccMain + cg * kChunk, a1);
          load_swizzled_row32(h_chunk, rloc, hv);
          tmem_ld_wait();
          const float* b = bias_s + bias_buf * 256 + cg * kChunk;
          gate_res_chunk(a0, a1, b, b + 128, hv, rg);
          store_swizzled_row32(h_chunk, rloc, hv);
        }
        if (cg & 1) { xch_s[(cg >> 1) * 256 + rloc * 2] = rg.pm; xch_s[(cg >> 1) * 256 + rloc * 2 + 1] = rg.pm2; }
        asm volatile("bar.sync 1, %0;" ::"n"(kChEpiThreads) : "memory");
        if (!(cg & 1) && ok && valid) {
          chan_merge_equal(rg.pm, rg.pm2, xch_s[(cg >> 1) * 256 + rloc * 2], xch_s[(cg >> 1) * 256 + rloc * 2 + 1],
                           static_cast<float>(kChunk));
          reinterpret_cast<float2*>(p.stats)[static_cast<size_t>(m) * G + (n_base / kStatCols) + (cg >> 1)] =
              make_float2(rg.pm, rg.pm2);
        }
        phase_end((1 << ACC_GATE) | (1 << ACC_MAIN));                    // sync base + 3 k + 2
      }

      // ---- step boundary: eps_hat, guidance, Eq. 3 update; then h and its partials for step t - 1
      sync_until(base + 3 * L);
      {
        const float ca = p.sched[t - 1], cb = p.sched[T + t - 1], cs = p.sched[2 * T + t - 1];
        for (int i = et; i < TB * kCPad; i += kChEpiThreads) {
          const int tok = tb * TB + (i >> 4), c = i & 15;
          float xn = 0.0f;
          if (ok && tok < p.R && c < p.C) {
            float e[2] = {0.0f, 0.0f};
            for (int rp = 0; rp < nrep; ++rp) {
              const float* src = p.epart + (static_cast<size_t>(tok + rp * p.R) * G) * kCPad + c;
              float acc = 0.0f;
              for (int n8 = 0; n8 < G; n8 += 8) {   // loads in batches, sums in group order
                float pv[8];
#pragma unroll
                for (int i8 = 0; i8 < 8; ++i8) pv[i8] = (n8 + i8 < G) ? __ldcg(src + (n8 + i8) * kCPad) : 0.0f;
#pragma unroll
                for (int i8 = 0; i8 < 8; ++i8) if (n8 + i8 < G) acc += pv[i8];
              }
              e[rp] = acc + p.bout[c];
            }
            const float eh = p.cfg ? cfg_combine(e[0], e[1], p.cfg_scale) : e[0];
            const size_t o = static_cast<size_t>(tok) * p.C + c;
            const float xo = x_s[i];
            const float mu = ddpm_mean(ca, xo, cb, eh);
            xn = ddpm_sample(mu, cs, p.eps[static_cast<size_t>(t - 1) * p.R * p.C + o]);
            if (t == 1 && j == 0) {
              p.mu1[o] = mu;
              if (p.x1) p.x1[o] = xo;
              if (p.sample_last && p.x0) p.x0[o] = xn;
            }
          }
          x_s[i] = xn;
        }
      }
      if (t == 1) break;
      bias_fetch(0);
      asm volatile("bar.sync 1, %0;" ::"n"(kChEpiThreads) : "memory");
      input_proj();
      phase_end(0);                                                      // sync base + 3 L + 1
      if (t >= 3) cond_vector(t - 2);   // into the buffer of s(t), which no CTA reads any more
    }
    if (!ok && lane == 0) ch_fail(p.err, DEV_ERR_EPI_WAIT, 0, 0);
    __syncwarp();
  }
  // no CTA leaves while a peer may still signal it
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive(); cluster_wait();
  if (warp == 1) tmem_dealloc(tmem_base, 512);
}

}  // namespace csd

