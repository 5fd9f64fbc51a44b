// GEMM kernels of the head: out-tile[128 x TN] = epilogue(A[M,K] * B[N,K]^T ...).
//   gemm_tc_kernel   : 16-bit operands on tcgen05 tensor cores, TMA-fed shared-memory ring, fp32
//                      accumulators in TMEM, warp-specialised (2 TMA warps / MMA warp / epilogue warps);
//                      TN = 64 or 128 output columns per CTA (64 when 128 would leave SMs idle).
//   gemm_simt_kernel : fp32 operands on plain FMA units (CSD_F32 heads), TN = 128.
// Accumulator layout, by template parameters (NSEG segments, MMA_N rows of B per k-step):
//   NSEG=1, MMA_N=TN   : acc0 = A0 * B0[tile rows]^T
//   NSEG=1, MMA_N=2*TN : B0 holds the AdaLN shift and scale rows interleaved in groups of 64
//                        (64 shift rows | 64 scale rows | next 64 shift rows | ...), one shared A:
//                        output column c pairs accumulator column (c/64)*128 + c%64 (shift) with
//                        the one 64 further (scale).
//   NSEG=2, MMA_N=TN   : acc0 = A0 * B0^T, acc1 = A1 * B1^T (AdaLN gate | second MLP layer).
#pragma once
#include "epilogue.cuh"
#include "ptx.cuh"

namespace csd {

constexpr int kBlockK = 64;  // bf16 elements per TMA box row = 128 bytes = one swizzle row
// Warp roles: warp 0 TMA (A), warp 1 MMA, then the epilogue warps, last warp TMA (B).  A tile has
// TN/32 column chunks x 4 TMEM lane quarters; the cheap epilogues of 128-wide tiles run 16 warps
// (one chunk per thread), everything else 8 warps (two chunks per thread, or one when TN = 64).
template <int EPI, int TN> struct TcWarps {
  static constexpr int kEpi = (TN >= 128 && (EPI == EPI_SILU_ACT || EPI == EPI_BIAS_F32)) ? 16 : 8;
  static constexpr int kThreads = (kEpi + 3) * 32;
  static constexpr int kChunksPerThread = (TN / kChunk) * 4 / kEpi;
};

enum DevErr : int { DEV_OK = 0, DEV_ERR_TMA_WAIT = 1, DEV_ERR_MMA_WAIT = 2, DEV_ERR_EPI_WAIT = 3 };

// PAIR: two CTAs of a cluster share one MMA (cta_group::2, M = 256): each holds its own 128 rows of A
// and half of the B rows, which cuts the shared-memory traffic per CTA and k-block.
template <int EPI, int MMA_N, int TN, bool PAIR> struct TcCfg {
  static constexpr bool kStageH = EPI == EPI_MOD || epi_is_modf<EPI>() || EPI == EPI_GATE_RES;
  // A stage holds kKps k-blocks of 64 elements (one TMA box per operand and k-block).  The kernels whose
  // MMAs are 128 wide use two: fewer barrier round trips per byte.
  static constexpr int kKps = ((EPI == EPI_SILU_ACT || EPI == EPI_GATE_RES) && MMA_N <= 128) ? 2 : 1;
  static constexpr int kABoxBytes = kTileM * kBlockK * 2;
  static constexpr int kBRows = PAIR ? MMA_N / 2 : MMA_N;    // rows of the B tile this CTA loads
  static constexpr int kBBoxBytes = kBRows * kBlockK * 2;
  static constexpr int kABytes = kKps * kABoxBytes;
  static constexpr int kBBytes = kKps * kBBoxBytes;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kHTileBytes = kTileM * TN * 4;        // fp32 h tile staged in shared memory
  static constexpr int kHBytes = kStageH ? kHTileBytes : 0;
  // 16-bit output tiles (SiLU and modulate epilogues) leave through shared memory and TMA stores: a thread owns a row,
  // so direct stores touch 32 lines per instruction, and such bursts hold up the TMA loads of the next tile's
  // mainloop.  The modulate epilogue reuses the h tile it has just read; the SiLU epilogue gets a buffer of its own.
  static constexpr bool kStagedOut = EPI == EPI_SILU_ACT || EPI == EPI_MOD;
  static constexpr int kOutBytes = EPI == EPI_SILU_ACT ? kTileM * TN * 2 : 0;
  static constexpr int kWoutBytes = epi_is_modf<EPI>() ? kTileM * epi_out_width<EPI>() * 4 : 0;   // Wout^T tile [TN][16 or 32], reused for [128 rows][..] partials
  static constexpr int kXchBytes = (EPI == EPI_GATE_RES || epi_is_modf<EPI>()) ? kTileM * 16 : 0;   // per-row exchange between column halves
  static constexpr int kMiscBytes = 2 * TN * 4 + kXchBytes;     // two bias slices + exchange
  static constexpr int kFixedBytes = 1024 + kHBytes + kOutBytes + kWoutBytes + kMiscBytes + 256;
  static constexpr int kStagesMax = (227 * 1024 - kFixedBytes) / kStageBytes;
  static constexpr int kStages = kStagesMax > 8 ? 8 : kStagesMax;
  static constexpr int kSmemBytes = kFixedBytes + kStages * kStageBytes;
};

// Reads 32 consecutive floats of row r from a [128 rows][128 bytes] tile that TMA wrote with the
// 128-byte swizzle (16-byte unit j of row r lives at unit j ^ (r & 7)).
__device__ __forceinline__ void load_swizzled_row32(const uint8_t* tile, int r, float* v) {
  const uint8_t* row = tile + r * 128;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float4 q = *reinterpret_cast<const float4*>(row + ((j ^ (r & 7)) << 4));
    v[4 * j] = q.x; v[4 * j + 1] = q.y; v[4 * j + 2] = q.z; v[4 * j + 3] = q.w;
  }
}

// The inverse: writes 32 floats of row r in the layout a TMA store with the 128-byte swizzle expects.
__device__ __forceinline__ void store_swizzled_row32(uint8_t* tile, int r, const float* v) {
  uint8_t* row = tile + r * 128;
#pragma unroll
  for (int j = 0; j < 8; ++j)
    *reinterpret_cast<float4*>(row + ((j ^ (r & 7)) << 4)) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
}

// Persistent over tiles: CTA b handles output tiles b, b + gridDim.x, ... (column tile fastest).  The
// shared-memory ring runs on across tiles; the accumulators are double-buffered in TMEM, so the
// epilogue of one tile overlaps the MMAs of the next.
template <int EPI, typename ACT, int NSEG, int MMA_N, int TN, int AB_FMT, bool PAIR>
__global__ void __launch_bounds__(TcWarps<EPI, TN>::kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
               const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmB1,
               const __grid_constant__ CUtensorMap tmH, const __grid_constant__ CUtensorMap tmOut, int nkb0, int nkb1, int dep_kb,
               int tiles_n, int tiles_total,
               EpiParams ep, int* err) {
  using Cfg = TcCfg<EPI, MMA_N, TN, PAIR>;
  constexpr int S = Cfg::kStages;
  constexpr int EW = TcWarps<EPI, TN>::kEpi, CPT = TcWarps<EPI, TN>::kChunksPerThread, kEpiThreads = EW * 32;
  constexpr int NC = TN / kChunk;               // column chunks per tile
  constexpr bool kPacked = (NSEG == 1) && (MMA_N == 2 * TN);
  constexpr int EPW = epi_out_width<EPI>();   // output-projection columns (EPI_MODF, EPI_MODF2)
  constexpr bool kTwoAcc = kPacked || NSEG == 2;
  constexpr uint32_t kAccCols = NSEG * MMA_N;   // 64, 128 or 256 columns per accumulator buffer
  constexpr uint32_t kTmemCols = 2 * kAccCols;  // two buffers: a power of two in [128, 512]
  static_assert(MMA_N == TN || kPacked, "MMA_N is TN or 2 TN");
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* stage_base = smem;
  uint8_t* h_s = smem + S * Cfg::kStageBytes;                    // NC chunks of [128 rows][128 B], swizzled
  uint8_t* out_s = h_s + Cfg::kHBytes;                           // SiLU epilogue: outgoing 16-bit tile, boxes of 64 columns
  float* wout_s = reinterpret_cast<float*>(out_s + Cfg::kOutBytes);
  float* bias_s = reinterpret_cast<float*>(out_s + Cfg::kOutBytes + Cfg::kWoutBytes);
  float* xch_s = bias_s + 2 * TN;                            // [128 rows][4] exchange between column halves
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(out_s + Cfg::kOutBytes + Cfg::kWoutBytes + Cfg::kMiscBytes);
  uint64_t* empty_bar = full_bar + S;
  uint64_t* tmem_full_bar = empty_bar + S;      // [2]
  uint64_t* tmem_empty_bar = tmem_full_bar + 2; // [2]
  uint64_t* h_bar = tmem_empty_bar + 2;
  uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(h_bar + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int KPS = Cfg::kKps;
  // from here on nkb0 / nkb1 / dep_kb / total_kb count stages of KPS k-blocks
  nkb0 /= KPS; nkb1 /= KPS; dep_kb /= KPS;
  const int total_kb = nkb0 + (NSEG == 2 ? nkb1 : 0);
  // Work unit index and count: a CTA, or a pair of CTAs (cluster ranks 0 = leader and 1).  With pairs
  // tiles_total counts pair tiles (two row tiles each) and the pair's CTAs take row tiles 2p and 2p+1.
  const int rank = PAIR ? static_cast<int>(cluster_ctarank()) : 0;
  const int unit = PAIR ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
  const int nunits = PAIR ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);
  const int my_tiles = (tiles_total - unit + nunits - 1) / nunits;

  // Once any kernel of this context has raised the error flag, later launches return at once
  // (a decision uniform over the block, and over the pair) so that a failure costs one bounded
  // wait, not one per launch.
  __shared__ int s_abort;
  if (threadIdx.x == 0) s_abort = *reinterpret_cast<volatile int*>(err);
  __syncthreads();
  if (PAIR) {
    cluster_arrive(); cluster_wait();               // the peer has published its flag
    int peer_abort = 0;
    if (threadIdx.x == 0) {
      const uint32_t pa = mapa_shared(smem_u32(&s_abort), static_cast<uint32_t>(rank ^ 1));
      asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(peer_abort) : "r"(pa) : "memory");
    }
    cluster_arrive(); cluster_wait();               // both have read before either may overwrite
    if (threadIdx.x == 0 && peer_abort != 0) s_abort = peer_abort;
    __syncthreads();
  }
  if (s_abort != 0) return;

  if (warp == 0 && lane == 0) {
    tma_prefetch_desc(&tmA0);
    tma_prefetch_desc(&tmB0);
    if (NSEG == 2) { tma_prefetch_desc(&tmA1); tma_prefetch_desc(&tmB1); }
    if (Cfg::kStageH) tma_prefetch_desc(&tmH);
    if (Cfg::kStagedOut) tma_prefetch_desc(&tmOut);
    for (int s = 0; s < S; ++s) { mbar_init(&full_bar[s], 2); mbar_init(&empty_bar[s], 1); }
    // a pair's accumulator buffer is released by the epilogues of both CTAs (to the leader's barrier)
    for (int i = 0; i < 2; ++i) { mbar_init(&tmem_full_bar[i], 1); mbar_init(&tmem_empty_bar[i], PAIR ? 2 : 1); }
    mbar_init(h_bar, 1);
    fence_mbar_init();
  }
  if (warp == 1) {
    if (PAIR) { tmem_alloc_pair(tmem_base_s, kTmemCols); tmem_relinquish_pair(); }
    else { tmem_alloc(tmem_base_s, kTmemCols); tmem_relinquish(); }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (PAIR) { cluster_arrive(); cluster_wait(); }   // the peer's barriers exist before anything signals them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_base_s;

  // Two TMA producers: one thread sustains only about one request per 240 clk, so the activation
  // tiles (A, warp 0) and the weight tiles (B, last warp) are requested by different warps; each arms
  // the stage's barrier with its own byte count.  Weights never depend on the preceding kernel; of
  // the activations only k-blocks >= dep_kb do (the A producer waits for it there, once), so the part
  // of the product that is independent of the preceding kernel overlaps with that kernel.
  auto produce = [&](const CUtensorMap* t0, const CUtensorMap* t1, uint32_t bytes, int off, bool is_a, int wait_kb) {
    bool ok = true;
    int it = 0;   // k-blocks issued so far over all tiles
    for (int i = 0; i < my_tiles && ok; ++i) {
      const int t = unit + i * nunits;
      const int tm = PAIR ? 2 * (t / tiles_n) + rank : t / tiles_n;
      const int crd = is_a ? tm * kTileM : (t % tiles_n) * MMA_N + rank * Cfg::kBRows;
      for (int kb = 0; kb < total_kb; ++kb, ++it) {
        const int s = it % S;
        if (i == 0 && kb == wait_kb) griddep_wait();
        if (it >= S && !mbar_wait(&empty_bar[s], ((it / S) & 1) ^ 1)) { atomicExch(err, DEV_ERR_TMA_WAIT); ok = false; break; }
        const CUtensorMap* tmap = (NSEG == 2 && kb >= nkb0) ? t1 : t0;
        const int kx = ((NSEG == 2 && kb >= nkb0) ? kb - nkb0 : kb) * KPS * kBlockK;
        uint8_t* dst = stage_base + s * Cfg::kStageBytes + off;
        if (PAIR) {
          // the leader's barrier counts the bytes of both CTAs; only the leader arms it
          if (rank == 0) mbar_arrive_expect_tx(&full_bar[s], 2 * bytes);
          const uint32_t lb = mapa_shared(smem_u32(&full_bar[s]), 0);
#pragma unroll
          for (int j = 0; j < KPS; ++j) tma_load_2d_pair(dst + j * (bytes / KPS), tmap, lb, kx + j * kBlockK, crd);
        } else {
          mbar_arrive_expect_tx(&full_bar[s], bytes);
#pragma unroll
          for (int j = 0; j < KPS; ++j) tma_load_2d(dst + j * (bytes / KPS), tmap, &full_bar[s], kx + j * kBlockK, crd);
        }
      }
    }
  };
  if (warp == 0) {            // activation tiles
    if (lane == 0) produce(&tmA0, &tmA1, Cfg::kABytes, 0, true, dep_kb);
    __syncwarp();
  } else if (warp == EW + 2) {    // weight tiles
    if (lane == 0) produce(&tmB0, &tmB1, Cfg::kBBytes, Cfg::kABytes, false, -1);
    __syncwarp();
  } else if (warp == 1) {
    if (rank == 0) {     // of a pair only the leader issues MMAs
      // The whole warp runs the loop and waits; one elected lane issues.  (Measured: a loop entered by a
      // single lane spends about 200 clk more per stage on the same waits, MMAs and commit.)
      const bool leader = elect_one();
      constexpr uint32_t idesc = umma_idesc_f16(MMA_N, AB_FMT, PAIR ? 256 : 128);
      bool ok = true;
      int it = 0;
      for (int i = 0; i < my_tiles && ok; ++i) {
        const int ab = i & 1;
        // the epilogue must have drained this accumulator buffer (tile i - 2)
        if (i >= 2 && !mbar_wait(&tmem_empty_bar[ab], ((i >> 1) - 1) & 1)) { if (leader) atomicExch(err, DEV_ERR_MMA_WAIT); ok = false; break; }
        tc_fence_after_sync();
        for (int kb = 0; kb < total_kb; ++kb, ++it) {
          const int s = it % S;
          if (!mbar_wait(&full_bar[s], (it / S) & 1)) { if (leader) atomicExch(err, DEV_ERR_MMA_WAIT); ok = false; break; }
          tc_fence_after_sync();
          if (leader) {
            const bool second = (NSEG == 2) && (kb >= nkb0);
            const int kk = second ? kb - nkb0 : kb;
            const uint32_t sa = smem_u32(stage_base + s * Cfg::kStageBytes);
            const uint32_t d = tmem_base + ab * kAccCols + (second ? MMA_N : 0);
#pragma unroll
            for (int j = 0; j < KPS; ++j) {
              const uint64_t da = umma_smem_desc_sw128(sa + j * Cfg::kABoxBytes);
              const uint64_t db = umma_smem_desc_sw128(sa + Cfg::kABytes + j * Cfg::kBBoxBytes);
#pragma unroll
              for (int k = 0; k < kBlockK / 16; ++k) {  // UMMA_K = 16 elements = 32 bytes = 2 descriptor units
                const uint32_t acc = (kk > 0 || j > 0 || k > 0) ? 1u : 0u;
                if (PAIR) umma_f16_pair(d, da + 2 * k, db + 2 * k, idesc, acc);
                else umma_f16(d, da + 2 * k, db + 2 * k, idesc, acc);
              }
            }
            if (PAIR) umma_commit_pair(&empty_bar[s]); else umma_commit(&empty_bar[s]);
          }
          __syncwarp();
        }
        if (ok && leader) { if (PAIR) umma_commit_pair(&tmem_full_bar[ab]); else umma_commit(&tmem_full_bar[ab]); }
        __syncwarp();
      }
    }
    __syncwarp();
  } else {
    // Epilogue: warp w may touch TMEM lanes [32 (w % 4), 32 (w % 4) + 32).  With 8 warps, warps 2..5
    // take column chunks 0 and 1 of the tile and warps 6..9 chunks 2 and 3 (one chunk each when the
    // tile is 64 wide); with 16 warps each group of four takes one chunk.
    const int et = threadIdx.x - 64;
    const int q = warp & 3, half = (warp - 2) >> 2;   // half = chunk group
    const int rloc = q * 32 + lane;
    // h, the LayerNorm partials and the right to overwrite this kernel's outputs come with the
    // completion of the preceding kernel.  Only then may the next kernel start its own early part
    // (at most one kernel runs ahead).
    // per-tile constants (biases, the Wout^T tile): not written by any kernel, so those of the first tile
    // are staged before the wait
    auto stage_consts = [&](int tile_n) {
      if (et < TN) {
        bias_s[et] = ep.bias0[tile_n * TN + et];
        bias_s[TN + et] = ep.bias1 ? ep.bias1[tile_n * TN + et] : 0.0f;
      }
      if (epi_is_modf<EPI>()) {
        const float4* src = reinterpret_cast<const float4*>(ep.wout_t + static_cast<size_t>(tile_n) * TN * EPW);
        float4* dst = reinterpret_cast<float4*>(wout_s);
#pragma unroll
        for (int j = 0; j < TN * EPW / 4 / kEpiThreads; ++j) dst[et + j * kEpiThreads] = src[et + j * kEpiThreads];
      }
    };
    stage_consts(unit % tiles_n);
    griddep_wait();
    if (et == 0) griddep_launch_dependents();
    bool ok = true;
    for (int i = 0; i < my_tiles; ++i) {
      const int t = unit + i * nunits;
      const int tile_n = t % tiles_n, tile_m = PAIR ? 2 * (t / tiles_n) + rank : t / tiles_n;
      const int ab = i & 1;
      const int m = tile_m * kTileM + rloc;
      const bool valid = m < ep.M;
      // every epilogue thread is done with the previous tile: its accumulator buffer, the h tile and
      // the per-tile constants may be replaced
      asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
      if (et == 0) {
        if (i >= 1) {
          if (PAIR) mbar_arrive_cluster(mapa_shared(smem_u32(&tmem_empty_bar[ab ^ 1]), 0));
          else mbar_arrive(&tmem_empty_bar[ab ^ 1]);
        }
        if (Cfg::kStagedOut && i >= 1) {
          // the previous tile's 16-bit output sits in shared memory (the modulate epilogue wrote it over the h tile)
          const int tp = unit + (i - 1) * nunits;
          const int pn = tp % tiles_n, pm = PAIR ? 2 * (tp / tiles_n) + rank : tp / tiles_n;
#pragma unroll
          for (int b = 0; b < TN / 64; ++b)
            tma_store_2d(&tmOut, (EPI == EPI_MOD ? h_s + 2 * b * (kTileM * 128) : out_s + b * (kTileM * 128)), pn * TN + b * 64, pm * kTileM);
          tma_store_commit();
          tma_store_wait_read();   // before this tile's h lands on it / the epilogue writes the next tile
        }
        if (EPI == EPI_GATE_RES && i >= 1) {
          // the previous tile's new h sits in the h tile (the threads that own its rows wrote it in place): TMA
          // stores instead of row-per-thread stores, which touch 32 rows per instruction
          const int tp = unit + (i - 1) * nunits;
          const int pn = tp % tiles_n, pm = PAIR ? 2 * (tp / tiles_n) + rank : tp / tiles_n;
#pragma unroll
          for (int c = 0; c < NC; ++c) tma_store_2d(&tmH, h_s + c * (kTileM * 128), pn * TN + c * kChunk, pm * kTileM);
          tma_store_commit();
          tma_store_wait_read();   // before the next h tile lands on it
        }
        if (Cfg::kStageH) {
          // requested before this thread block's further pipeline traffic queues up behind it: ordinary
          // loads issued while the pipeline saturates the SM's shared-memory port take thousands of cycles
          mbar_arrive_expect_tx(h_bar, Cfg::kHTileBytes);
#pragma unroll
          for (int c = 0; c < NC; ++c)
            tma_load_2d(h_s + c * (kTileM * 128), &tmH, h_bar, tile_n * TN + c * kChunk, tile_m * kTileM);
        }
      }
      if (i > 0) stage_consts(tile_n);
      RowState rs;
      if (valid) epi_row_begin<EPI>(ep, m, rs);
      asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");   // biases and the Wout^T tile are in place
      if (ok) ok = mbar_wait(&tmem_full_bar[ab], (i >> 1) & 1);
      if (ok && Cfg::kStageH) ok = mbar_wait(h_bar, i & 1);
      if (!ok) atomicExch(err, DEV_ERR_EPI_WAIT);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        tc_fence_after_sync();
        const uint32_t trow = tmem_base + ab * kAccCols + (static_cast<uint32_t>(q * 32) << 16);
#pragma unroll
        for (int ci = 0; ci < CPT; ++ci) {
          const int c = CPT * half + ci;
          float a0[kChunk], a1[kChunk], hv[kChunk];
          const int col0 = kPacked ? (c >> 1) * 128 + (c & 1) * kChunk : c * kChunk;   // first accumulator
          tmem_ld32(trow + col0, a0);
          if (kTwoAcc) tmem_ld32(trow + col0 + (kPacked ? kStatCols : TN), a1);
          if (Cfg::kStageH) load_swizzled_row32(h_s + c * (kTileM * 128), rloc, hv);
          tmem_ld_wait();
          float efirst[EPW];
          if (epi_is_modf<EPI>() && ci == 1) {
#pragma unroll
            for (int e = 0; e < EPW; ++e) { efirst[e] = rs.eacc[e]; rs.eacc[e] = 0.0f; }
          }
          if (EPI == EPI_GATE_RES) {
            gate_res_chunk(a0, a1, bias_s + c * kChunk, bias_s + TN + c * kChunk, hv, rs);
            store_swizzled_row32(h_s + c * (kTileM * 128), rloc, hv);   // in place; leaves by TMA store
          } else if (Cfg::kStagedOut) {
            if (EPI == EPI_SILU_ACT) {
#pragma unroll
              for (int j = 0; j < kChunk; ++j) a0[j] = silu_t<true>(a0[j] + bias_s[c * kChunk + j]);
            } else
              modulate_chunk(a0, a1, bias_s + c * kChunk, bias_s + TN + c * kChunk, hv, rs);
            // 64 bytes of row rloc in box c / 2 (TMA's 128-byte swizzle); the modulate epilogue writes over the h it read
            uint8_t* row = (EPI == EPI_MOD ? h_s + 2 * (c >> 1) * (kTileM * 128) : out_s + (c >> 1) * (kTileM * 128)) + rloc * 128;
            __align__(16) ACT o[kChunk];
#pragma unroll
            for (int j = 0; j < kChunk; ++j) o[j] = to_act<ACT>(a0[j]);
#pragma unroll
            for (int u = 0; u < 4; ++u)
              *reinterpret_cast<uint4*>(row + ((((c & 1) * 4 + u) ^ (rloc & 7)) << 4)) = reinterpret_cast<const uint4*>(o)[u];
          } else if (valid)
            epi_chunk<EPI, ACT, true>(ep, m, tile_n * TN + c * kChunk, a0, a1, bias_s + c * kChunk,
                                      bias_s + TN + c * kChunk, hv, rs, wout_s + c * kChunk * EPW);
          if (epi_is_modf<EPI>() && ci == 1) {
#pragma unroll
            for (int e = 0; e < EPW; ++e) rs.eacc[e] = efirst[e] + rs.eacc[e];
          }
        }
        if (EPI == EPI_GATE_RES || Cfg::kStagedOut) fence_proxy_async_smem();
        tc_fence_before_sync();   // orders the TMEM reads before the barrier that releases the buffer
      }
      if (EPI == EPI_GATE_RES) {
        // one (mean, M2) partial per row and 64-column group
        if (CPT == 2) {            // TN = 128: this thread's two chunks are one group
          if (ok && valid) store_group_stats(ep, m, tile_n * 2 + half, rs.pm, rs.pm2);
        } else {                   // TN = 64: chunk 1 (warps 6..9) is merged into chunk 0 (warps 2..5)
          if (half == 1) { xch_s[rloc * 4] = rs.pm; xch_s[rloc * 4 + 1] = rs.pm2; }
          asm volatile("bar.sync 1, 256;" ::: "memory");
          if (half == 0 && ok && valid) {
            chan_merge_equal(rs.pm, rs.pm2, xch_s[rloc * 4], xch_s[rloc * 4 + 1], static_cast<float>(kChunk));
            store_group_stats(ep, m, tile_n, rs.pm, rs.pm2);
          }
        }
      }
      if (epi_is_modf<EPI>()) {
        // one eps partial per row and 64-column group, always formed as (chunk sum) + (next chunk sum) so
        // that both tile widths give the same bits
        if (CPT == 2) {            // TN = 128: this thread's two chunks are one group
          if (ok && valid) epi_row_end<EPI>(ep, m, tile_n * 2 + half, rs);
        } else {                   // TN = 64: chunk 1 (warps 6..9) is added to chunk 0 (warps 2..5)
          asm volatile("bar.sync 1, 256;" ::: "memory");   // every thread is done reading the Wout^T tile
          float* part = wout_s;                            // [128 rows][EPW]
          if (half == 1 && ok) {
#pragma unroll
            for (int c = 0; c < EPW; ++c) part[rloc * EPW + c] = rs.eacc[c];
          }
          asm volatile("bar.sync 1, 256;" ::: "memory");
          if (half == 0 && ok && valid) {
#pragma unroll
            for (int c = 0; c < EPW; ++c) rs.eacc[c] += part[rloc * EPW + c];
            epi_row_end<EPI>(ep, m, tile_n, rs);
          }
        }
      }
    }
    if (Cfg::kStagedOut) {
      // the last tile's output
      asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
      if (et == 0 && ok) {
        const int tp = unit + (my_tiles - 1) * nunits;
        const int pn = tp % tiles_n, pm = PAIR ? 2 * (tp / tiles_n) + rank : tp / tiles_n;
#pragma unroll
        for (int b = 0; b < TN / 64; ++b)
          tma_store_2d(&tmOut, (EPI == EPI_MOD ? h_s + 2 * b * (kTileM * 128) : out_s + b * (kTileM * 128)), pn * TN + b * 64, pm * kTileM);
        tma_store_commit();
      }
      if (et == 0) tma_store_wait_all();
    }
    if (EPI == EPI_GATE_RES) {
      // the last tile's new h
      asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
      if (et == 0 && ok) {
        const int tp = unit + (my_tiles - 1) * nunits;
        const int pn = tp % tiles_n, pm = PAIR ? 2 * (tp / tiles_n) + rank : tp / tiles_n;
#pragma unroll
        for (int c = 0; c < NC; ++c) tma_store_2d(&tmH, h_s + c * (kTileM * 128), pn * TN + c * kChunk, pm * kTileM);
        tma_store_commit();
      }
      if (et == 0) tma_store_wait_all();
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (PAIR) { cluster_arrive(); cluster_wait(); }   // neither CTA leaves while the pair's MMAs or signals may touch it
  if (warp == 1) { if (PAIR) tmem_dealloc_pair(tmem_base, kTmemCols); else tmem_dealloc(tmem_base, kTmemCols); }
}

// ------------------------------------------------------------------ fp32 FMA path
constexpr int kSimtRows = 32;
constexpr int kSimtBK = 32;

template <int EPI, int NSEG, int MMA_N>
__global__ void __launch_bounds__(128)
gemm_simt_kernel(const float* __restrict__ A0, int lda0, const float* __restrict__ B0, int ldb0, int K0,
                 const float* __restrict__ A1, int lda1, const float* __restrict__ B1, int ldb1, int K1,
                 EpiParams ep) {
  __shared__ float As[kSimtRows][kSimtBK + 1];
  __shared__ float Bs[MMA_N][kSimtBK + 1];
  constexpr int EPW = epi_out_width<EPI>();
  // the 16-column Wout^T tile is staged in shared memory; the 32-column one would not fit beside the operand tiles
  // and is read through L1 instead
  constexpr bool kStageWout = EPI == EPI_MODF;
  __shared__ float wout_s[kStageWout ? kTileN * EPW : 1];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int tile_n = blockIdx.x, m0 = blockIdx.y * kSimtRows;
  const int m = m0 + lane;
  if (kStageWout) {
    const float* src = ep.wout_t + static_cast<size_t>(tile_n) * kTileN * EPW;
    for (int i = threadIdx.x; i < kTileN * EPW; i += 128) wout_s[i] = src[i];
  }
  float acc0[kChunk], acc1[kChunk];
#pragma unroll
  for (int j = 0; j < kChunk; ++j) { acc0[j] = 0.0f; acc1[j] = 0.0f; }
#pragma unroll 1
  for (int seg = 0; seg < NSEG; ++seg) {
    const float* A = seg ? A1 : A0;
    const float* B = seg ? B1 : B0;
    const int lda = seg ? lda1 : lda0, ldb = seg ? ldb1 : ldb0, K = seg ? K1 : K0;
    const int brow0 = tile_n * MMA_N;
#pragma unroll 1
    for (int k0 = 0; k0 < K; k0 += kSimtBK) {
      for (int i = threadIdx.x; i < kSimtRows * kSimtBK; i += 128) {
        const int r = i / kSimtBK, c = i % kSimtBK;
        As[r][c] = (m0 + r < ep.M) ? A[static_cast<size_t>(m0 + r) * lda + k0 + c] : 0.0f;
      }
      for (int i = threadIdx.x; i < MMA_N * kSimtBK; i += 128) {
        const int r = i / kSimtBK, c = i % kSimtBK;
        Bs[r][c] = B[static_cast<size_t>(brow0 + r) * ldb + k0 + c];
      }
      __syncthreads();
#pragma unroll 4
      for (int k = 0; k < kSimtBK; ++k) {
        const float a = As[lane][k];
        if constexpr (MMA_N == 256) {
#pragma unroll
          for (int j = 0; j < kChunk; ++j) {
            acc0[j] = fmaf(a, Bs[(warp >> 1) * 128 + (warp & 1) * kChunk + j][k], acc0[j]);
            acc1[j] = fmaf(a, Bs[(warp >> 1) * 128 + (warp & 1) * kChunk + kStatCols + j][k], acc1[j]);
          }
        } else {
          if (seg == 0) {
#pragma unroll
            for (int j = 0; j < kChunk; ++j) acc0[j] = fmaf(a, Bs[warp * kChunk + j][k], acc0[j]);
          } else {
#pragma unroll
            for (int j = 0; j < kChunk; ++j) acc1[j] = fmaf(a, Bs[warp * kChunk + j][k], acc1[j]);
          }
        }
      }
      __syncthreads();
    }
  }
  // This thread owns chunk `warp` of the tile only; EPI_MODF partials are therefore per chunk
  // and summed below through shared memory in chunk order.
  RowState rs;
  if (m < ep.M) {
    const int n0 = tile_n * kTileN + warp * kChunk;
    float hv[kChunk];
    epi_row_begin<EPI>(ep, m, rs);
    if (epi_reads_h<EPI>()) load_chunk_f32(ep.h + static_cast<size_t>(m) * ep.ldo + n0, hv);
    epi_chunk<EPI, float, false>(ep, m, n0, acc0, acc1, ep.bias0 + n0, ep.bias1 ? ep.bias1 + n0 : ep.bias0 + n0, hv, rs,
                                 kStageWout ? wout_s + warp * kChunk * EPW
                                            : ep.wout_t + (static_cast<size_t>(tile_n) * kTileN + warp * kChunk) * EPW);
  }
  if constexpr (EPI == EPI_GATE_RES) {
    float* scr = &Bs[0][0];  // reused as [4 chunks][32 rows][4]: chunks (0,1) and (2,3) form the 64-column groups
    __syncthreads();
    if (m < ep.M && (warp & 1)) { scr[(warp * kSimtRows + lane) * 4] = rs.pm; scr[(warp * kSimtRows + lane) * 4 + 1] = rs.pm2; }
    __syncthreads();
    if (m < ep.M && !(warp & 1)) {
      chan_merge_equal(rs.pm, rs.pm2, scr[((warp + 1) * kSimtRows + lane) * 4], scr[((warp + 1) * kSimtRows + lane) * 4 + 1],
                       static_cast<float>(kChunk));
      store_group_stats(ep, m, tile_n * 2 + (warp >> 1), rs.pm, rs.pm2);
    }
  }
  if constexpr (epi_is_modf<EPI>()) {
    float* scr = &Bs[0][0];  // reused as [4 chunks][32 rows][EPW]
    __syncthreads();
    if (m < ep.M) {
#pragma unroll
      for (int c = 0; c < EPW; ++c) scr[(warp * kSimtRows + lane) * EPW + c] = rs.eacc[c];
    }
    __syncthreads();
    if (warp == 0 && m < ep.M) {
#pragma unroll
      for (int c = 0; c < EPW; ++c) {
        float v = 0.0f;
        for (int w = 0; w < 4; ++w) v += scr[(w * kSimtRows + lane) * EPW + c];
        rs.eacc[c] = v;
      }
      epi_row_end<EPI>(ep, m, tile_n, rs);
    }
  }
}

}  // namespace csd
