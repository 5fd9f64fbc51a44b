// Two kernels per residual block instead of three, for grids of one wave (the launch-latency regime).
//
// The block is  u = LN(h)(1 + scale) + shift;  v = SiLU(W1 u + b1);  h += gate . (W2 v + b2)  with
// (shift, scale, gate) = Wada s + bada.  LayerNorm folds into the first layer's epilogue:
//     W1 u + b1 = rstd [ (h . (1 + scale)) W1^T  -  mean ((1 + scale) W1^T) ]  +  shift W1^T + b1
// and the two row vectors in s are again products of s with weights fused once per head,
//     (1 + scale) W1^T = s (W1 Wscale)^T + W1 (1 + bscale)  =: P1 + c1,
//     shift W1^T + b1  = s (W1 Wshift)^T + W1 bshift + b1   =: P2 + c2.
// So the kernel that updates h can hand the next block  a' = h . (1 + scale_next)  directly, and the separate
// "modulate" kernel (a full kernel on the chain of dependent launches, although only its epilogue waits)
// disappears:
//   fold_kernel<KIND_GATE> : acc(gate | scale_next) = s [Wg_k | Wscale_{k+1}]^T  (early, N = 256 packed),
//                            acc_main = v W2_k^T;  h += (gate + bg)(acc_main + b2), LayerNorm partials of the new h,
//                            a' = h (1 + scale_next + bscale_next)
//   fold_kernel<KIND_W1>   : acc(P1 | P2) = s [W1 Wscale | W1 Wshift]^T          (early, N = 256 packed),
//                            acc_main = a' W1_k^T;  v = SiLU(rstd (acc_main - mean (P1 + c1)) + P2 + c2)
// The early products depend only on s and overlap the preceding kernel (programmatic dependent launch).
// One tile per CTA (128 x 128), a 192 KB TMA ring, three TMEM accumulators, three TMA warps, one MMA warp,
// eight epilogue warps (one row x 64 columns per thread).
// PAIR: two CTAs of a cluster (row tiles 2p and 2p + 1 of one column tile) share every MMA (cta_group::2, M = 256):
// each loads its own rows of the activations and half of the weight rows, so a k-block of the dependent product
// costs a CTA 24 KB of shared-memory traffic instead of 32 KB and the ring holds four two-k-block stages instead of
// three: the product that the preceding kernel gates is bound by what the ring keeps in flight, not by the MMAs.
#pragma once
#include "gemm.cuh"
#include "rowops.cuh"

namespace csd {

constexpr int kChSlotBytes = 32768;   // ring slot: [A tile 16 KB | B tile 16 KB]

enum FoldKind : int { FOLD_W1 = 0, FOLD_GATE = 1 };

template <int KIND> struct FoldCfg {
  static constexpr int kSlots = 6;
  static constexpr int kHBytes = 0;
  static constexpr int kBiasBytes = 3 * 128 * 4;
  static constexpr int kSmemBytes = 1024 + kSlots * kChSlotBytes + kHBytes + kBiasBytes + 256;
};
constexpr int kFoldEpiWarps = 8;
constexpr int kFoldThreads = (kFoldEpiWarps + 4) * 32;   // + TMA activations (two warps), MMA, TMA weights
constexpr uint32_t kFoldAccPacked = 0, kFoldAccMain = 256;

struct FoldParams {
  int M, W;
  const float *c0, *c1, *c2;   // FOLD_W1: c1, c2, unused;  FOLD_GATE: gate bias, second-layer bias, next scale bias
  const float* stats_in;       // FOLD_W1: LayerNorm partials of h [M, W/64, 2]
  float* stats_out;            // FOLD_GATE: partials of the new h
  float* h;                    // FOLD_GATE: [M, W] read-modify-write
  void* out;                   // FOLD_W1: v;  FOLD_GATE: a' = h (1 + scale_next)
  int* err;
};

template <typename ACT, int AB_FMT, int KIND, bool PAIR>
__global__ void __launch_bounds__(kFoldThreads, 1)
fold_kernel(const __grid_constant__ CUtensorMap tmS, const __grid_constant__ CUtensorMap tmWp,
            const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
            const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmHst, int tiles_n,
            const FoldParams p) {
  using Cfg = FoldCfg<KIND>;
  // Ring stages.  Alone: three of 64 KB; early product [A 16 KB | packed 256-row weight tile 32 KB], dependent product two
  // k-blocks [A 16 KB | B 16 KB] each.  PAIR: four of 48 KB; early [A 16 KB | this CTA's 128 packed weight rows 16 KB],
  // dependent [A, A | this CTA's 64 weight rows 8 KB, 8 KB].
  constexpr int S = Cfg::kSlots, SP = PAIR ? 4 : 3, kPairBytes = PAIR ? 49152 : 2 * kChSlotBytes;
  constexpr int kDepA = PAIR ? 16384 : kChSlotBytes;          // dependent stage: distance between the two A boxes
  constexpr int kDepB0 = PAIR ? 32768 : 16384;                // first B box
  constexpr int kDepB = PAIR ? 8192 : kChSlotBytes;           // distance between the two B boxes
  static_assert(SP * kPairBytes == S * kChSlotBytes, "the ring is 192 KB either way");
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* ring = smem;
  float* bias_s = reinterpret_cast<float*>(ring + S * kChSlotBytes);   // [3][128]
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(bias_s + 384);
  uint64_t* empty_bar = full_bar + S;
  uint64_t* acc_full = empty_bar + S;    // [2]: packed, main
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(acc_full + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int W = p.W, nkb = W / kBlockK;
  const int rank = PAIR ? static_cast<int>(cluster_ctarank()) : 0;
  const int unit = PAIR ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
  const int tile_n = unit % tiles_n, tile_m = PAIR ? 2 * (unit / tiles_n) + rank : unit / tiles_n;
  const int n_base = tile_n * kTileN, row0 = tile_m * kTileM;

  const bool run = *reinterpret_cast<const volatile int*>(p.err) == 0;
  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmS); tma_prefetch_desc(&tmWp); tma_prefetch_desc(&tmA); tma_prefetch_desc(&tmW);
    tma_prefetch_desc(&tmOut);
    if (KIND == FOLD_GATE) tma_prefetch_desc(&tmHst);
    for (int s = 0; s < SP; ++s) { mbar_init(&full_bar[s], 3); mbar_init(&empty_bar[s], 1); }
    mbar_init(&acc_full[0], 1); mbar_init(&acc_full[1], 1);
    fence_mbar_init();
  }
  if (warp == 1) {
    if (PAIR) { tmem_alloc_pair(tmem_base_s, 512); tmem_relinquish_pair(); }
    else { tmem_alloc(tmem_base_s, 512); tmem_relinquish(); }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (PAIR) { cluster_arrive(); cluster_wait(); }   // the peer's barriers exist before anything signals them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_base_s;

  if (run && (warp == 0 || warp >= kFoldEpiWarps + 2)) {
    // ------------------------------------------------------------------ TMA requests: activations (warp 0 and, for the second
    // k-block of a dependent pair, the last warp: one thread sustains about one request per 300 clk), weights
    const bool is_a = warp != kFoldEpiWarps + 2;
    const bool second = warp == kFoldEpiWarps + 3;
    const bool leader = elect_one();
    bool ok = true;
    int it = 0;
    // The ring is used in pairs of slots (64 KB) with one full / empty barrier per pair: one barrier round trip
    // per k-block of the 256-wide early product and per two k-blocks of the 128-wide dependent one.
    auto pair_free = [&](int c) {   // c: pair counter
      if (ok && c >= SP) { ok = ch_wait<false>(&empty_bar[c % SP], ((c / SP) & 1) ^ 1, p.err); if (!ok && leader) ch_fail(p.err, DEV_ERR_TMA_WAIT, 2, c); }
    };
    // A pair's loads are all credited to the leader's barrier, which only the leader's producers arm (with the bytes
    // of both CTAs); the peer's producers only request.
    auto arm = [&](uint64_t* bar, uint32_t bytes) { if (!PAIR) mbar_arrive_expect_tx(bar, bytes); else if (rank == 0) mbar_arrive_expect_tx(bar, 2 * bytes); };
    auto load = [&](uint8_t* dst, const CUtensorMap* tm, uint64_t* bar, int x, int y) {
      if (PAIR) tma_load_2d_pair(dst, tm, mapa_shared(smem_u32(bar), 0), x, y); else tma_load_2d(dst, tm, bar, x, y);
    };
    // early product
    for (int kb = 0; kb < nkb && ok; ++kb, ++it) {
      pair_free(it);
      if (ok && leader) {
        const int s = it % SP;
        if (second) { if (rank == 0) mbar_arrive(&full_bar[s]); }
        else {
          arm(&full_bar[s], is_a ? 16384 : (PAIR ? 16384 : 32768));
          load(ring + s * kPairBytes + (is_a ? 0 : 16384), is_a ? &tmS : &tmWp, &full_bar[s], kb * kBlockK,
               is_a ? row0 : 2 * n_base + rank * 128);
        }
      }
      __syncwarp();
    }
    if (is_a) griddep_wait();            // the dependent operand is written by the preceding kernel
    // dependent product: two k-blocks per stage
    for (int kb = 0; kb < nkb && ok; kb += 2, ++it) {
      pair_free(it);
      if (ok && leader) {
        const int s = it % SP;
        if (is_a) {
          const int jj = second ? 1 : 0;
          arm(&full_bar[s], 16384);
          load(ring + s * kPairBytes + jj * kDepA, &tmA, &full_bar[s], (kb + jj) * kBlockK, row0);
        } else {
          arm(&full_bar[s], PAIR ? 16384 : 32768);
#pragma unroll
          for (int jj = 0; jj < 2; ++jj)
            load(ring + s * kPairBytes + kDepB0 + jj * kDepB, &tmW, &full_bar[s], (kb + jj) * kBlockK, n_base + rank * 64);
        }
      }
      __syncwarp();
    }
  } else if (run && warp == 1 && rank == 0) {
    // ------------------------------------------------------------------ MMA issue (of a pair, the leader's)
    const bool leader = elect_one();
    constexpr uint32_t idesc128 = umma_idesc_f16(128, AB_FMT, PAIR ? 256 : 128), idesc256 = umma_idesc_f16(256, AB_FMT, PAIR ? 256 : 128);
    auto mma = [&](uint32_t d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
      if (PAIR) umma_f16_pair(d, da, db, idesc, acc); else umma_f16(d, da, db, idesc, acc);
    };
    auto commit = [&](uint64_t* bar) { if (PAIR) umma_commit_pair(bar); else umma_commit(bar); };
    bool ok = true;
    int it = 0;
    for (int kb = 0; kb < nkb && ok; ++kb, ++it) {
      const int s = it % SP;
      ok = ch_wait<false>(&full_bar[s], (it / SP) & 1, p.err);
      if (!ok) { if (leader) ch_fail(p.err, DEV_ERR_MMA_WAIT, 7, it); break; }
      tc_fence_after_sync();
      if (leader) {
        const uint32_t sa = smem_u32(ring + s * kPairBytes);
        const uint64_t da = umma_smem_desc_sw128(sa), db = umma_smem_desc_sw128(sa + 16384);
#pragma unroll
        for (int k = 0; k < kBlockK / 16; ++k) mma(tmem_base + kFoldAccPacked, da + 2 * k, db + 2 * k, idesc256, (kb > 0 || k > 0) ? 1u : 0u);
        commit(&empty_bar[s]);
      }
      __syncwarp();
    }
    if (ok && leader) commit(&acc_full[0]);
    __syncwarp();
    // dependent product: two k-blocks per barrier round trip
    for (int kb = 0; kb < nkb && ok; kb += 2, ++it) {
      const int s = it % SP;
      ok = ch_wait<false>(&full_bar[s], (it / SP) & 1, p.err);
      if (!ok) { if (leader) ch_fail(p.err, DEV_ERR_MMA_WAIT, 6, it); break; }
      tc_fence_after_sync();
      if (leader) {
#pragma unroll
        for (int jj = 0; jj < 2; ++jj) {
          const uint32_t sa = smem_u32(ring + s * kPairBytes);
          const uint64_t da = umma_smem_desc_sw128(sa + jj * kDepA), db = umma_smem_desc_sw128(sa + kDepB0 + jj * kDepB);
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k) mma(tmem_base + kFoldAccMain, da + 2 * k, db + 2 * k, idesc128, (kb > 0 || jj > 0 || k > 0) ? 1u : 0u);
        }
        commit(&empty_bar[s]);
      }
      __syncwarp();
    }
    if (ok && leader) commit(&acc_full[1]);
    __syncwarp();
  } else if (run && warp >= 2 && warp < kFoldEpiWarps + 2) {
    // ------------------------------------------------------------------ epilogue: one row, two 32-column chunks of one 64-column group per thread
    constexpr int kEpiThreads = kFoldEpiWarps * 32;
    const int et = static_cast<int>(threadIdx.x) - 64;
    const int q = warp & 3, half = (warp - 2) >> 2;
    const int rloc = q * 32 + lane;
    const int m = row0 + rloc;
    const bool valid = m < p.M;
    const uint32_t trow = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    bool ok = true;
    auto bar_wait = [&](uint64_t* bar, int site) {
      int w = 1;
      if (ok && lane == 0) { w = ch_wait<false>(bar, 0, p.err) ? 1 : 0; if (!w) ch_fail(p.err, DEV_ERR_EPI_WAIT, site, 0); }
      w = __shfl_sync(0xffffffffu, w, 0);
      if (!w) ok = false;
    };
    // constants first: no kernel writes them
    if (et < 128) {
      bias_s[et] = p.c0[n_base + et];
      bias_s[128 + et] = p.c1[n_base + et];
      bias_s[256 + et] = p.c2 ? p.c2[n_base + et] : 0.0f;
    }
    griddep_wait();
    if (et == 0) griddep_launch_dependents();   // (letting the next kernel start before this wait was measured slower)
    float hv2[2][kChunk];
    if (KIND == FOLD_GATE) {
      // h of this thread's 64 columns, read past L1 (its writer may have overlapped this kernel's start)
#pragma unroll
      for (int ci = 0; ci < 2; ++ci) {
        const float4* src = reinterpret_cast<const float4*>(p.h + static_cast<size_t>(valid ? m : 0) * W + n_base + (2 * half + ci) * kChunk);
#pragma unroll
        for (int i = 0; i < kChunk / 4; ++i) {
          const float4 v4 = __ldcg(src + i);
          hv2[ci][4 * i] = v4.x; hv2[ci][4 * i + 1] = v4.y; hv2[ci][4 * i + 2] = v4.z; hv2[ci][4 * i + 3] = v4.w;
        }
      }
    }
    // The outputs leave through shared memory and TMA stores: a thread owns a row, so direct stores would touch 32
    // rows per instruction, 16 bytes each (measured: they, not the arithmetic, set the epilogue's length).  The ring
    // is free once the last MMA has completed: 16-bit tile in two boxes of 64 columns at its start, fp32 h behind.
    auto stage_act = [&](int c, const float* v) {
      uint8_t* row = ring + (c >> 1) * (kTileM * 128) + rloc * 128;
      ACT o[kChunk];
#pragma unroll
      for (int j = 0; j < kChunk; ++j) o[j] = to_act<ACT>(v[j]);
#pragma unroll
      for (int i = 0; i < 4; ++i)
        *reinterpret_cast<uint4*>(row + ((((c & 1) * 4 + i) ^ (rloc & 7)) << 4)) = reinterpret_cast<const uint4*>(o)[i];
    };
    RowState rs;
    rs.mean = 0.0f; rs.rstd = 0.0f; rs.pm = 0.0f; rs.pm2 = 0.0f; rs.pn = 0.0f;
    if (KIND == FOLD_W1 && valid) row_stats<true>(p.stats_in, m, W, rs.mean, rs.rstd);
    asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");   // constants are in place
    bar_wait(&acc_full[0], 3);
    bar_wait(&acc_full[1], 4);
    tc_fence_after_sync();
    if (ok) {
#pragma unroll
      for (int ci = 0; ci < 2; ++ci) {
        const int c = 2 * half + ci;                                  // 32-column chunk of the tile
        float a0[kChunk], a1[kChunk], am[kChunk];
        const uint32_t colp = kFoldAccPacked + (c >> 1) * 128 + (c & 1) * kChunk;
        tmem_ld32(trow + colp, a0);                                   // first packed product (P1 / gate)
        tmem_ld32(trow + colp + kStatCols, a1);                       // second packed product (P2 / next scale)
        tmem_ld32(trow + kFoldAccMain + c * kChunk, am);
        tmem_ld_wait();
        if (KIND == FOLD_W1) {
          const float* k1 = bias_s + c * kChunk;
          const float* k2 = bias_s + 128 + c * kChunk;
#pragma unroll
          for (int j = 0; j < kChunk; ++j) {
            const float t1 = __fsub_rn(am[j], __fmul_rn(rs.mean, __fadd_rn(a0[j], k1[j])));
            am[j] = silu_t<true>(fmaf(rs.rstd, t1, __fadd_rn(a1[j], k2[j])));
          }
          stage_act(c, am);
        } else {
          float* hv = hv2[ci];
          gate_res_chunk(a0, am, bias_s + c * kChunk, bias_s + 128 + c * kChunk, hv, rs);
          store_swizzled_row32(ring + 32768 + c * (kTileM * 128), rloc, hv);   // new h, one fp32 box per chunk
          const float* ks = bias_s + 256 + c * kChunk;
#pragma unroll
          for (int j = 0; j < kChunk; ++j) hv[j] = __fmul_rn(hv[j], __fadd_rn(1.0f, __fadd_rn(a1[j], ks[j])));
          stage_act(c, hv);
        }
      }
      if (KIND == FOLD_GATE && valid)
        reinterpret_cast<float2*>(p.stats_out)[static_cast<size_t>(m) * (W / kStatCols) + tile_n * 2 + half] = make_float2(rs.pm, rs.pm2);
    }
    fence_proxy_async_smem();
    asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
    if (et == 0 && ok) {
      tma_store_2d(&tmOut, ring, n_base, row0);
      tma_store_2d(&tmOut, ring + kTileM * 128, n_base + 64, row0);
      if (KIND == FOLD_GATE) {
#pragma unroll
        for (int c = 0; c < 4; ++c) tma_store_2d(&tmHst, ring + 32768 + c * (kTileM * 128), n_base + c * kChunk, row0);
      }
      tma_store_commit();
      tma_store_wait_all();
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (PAIR) { cluster_arrive(); cluster_wait(); }   // neither CTA leaves while the pair's MMAs or signals may touch it
  if (warp == 1) { if (PAIR) tmem_dealloc_pair(tmem_base, 512); else tmem_dealloc(tmem_base, 512); }
}

// C[n, i] = sum_j A[n, j] B[j, i], all [W, W] fp32 row-major: the once-per-head products W1 Wscale, W1 Wshift.
__global__ void __launch_bounds__(256) square_matmul_kernel(const float* __restrict__ A, const float* __restrict__ B,
                                                            float* __restrict__ C, int W) {
  __shared__ float As[32][33], Bs[32][33];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;     // 32 x 8 threads, 4 rows each
  const int n0 = blockIdx.y * 32, i0 = blockIdx.x * 32;
  float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
  for (int j0 = 0; j0 < W; j0 += 32) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      As[ty * 4 + r][tx] = A[static_cast<size_t>(n0 + ty * 4 + r) * W + j0 + tx];
      Bs[ty * 4 + r][tx] = B[static_cast<size_t>(j0 + ty * 4 + r) * W + i0 + tx];
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const float b = Bs[j][tx];
#pragma unroll
      for (int r = 0; r < 4; ++r) acc[r] = fmaf(As[ty * 4 + r][j], b, acc[r]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) C[static_cast<size_t>(n0 + ty * 4 + r) * W + i0 + tx] = acc[r];
}

}  // namespace csd
