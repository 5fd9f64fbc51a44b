// Fused epilogues of the head's GEMMs.  One thread owns one output row and walks its 64- or
// 128-column output tile in chunks of 32 columns; the same code serves the tcgen05 kernel (chunks read from
// TMEM) and the fp32 FMA kernel (chunks held in registers).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace csd {

constexpr int kTileM = 128;   // rows per tensor-core tile
constexpr int kTileN = 128;   // output columns per tile of the fp32 FMA kernel (the tcgen05 kernel: 64 or 128)
constexpr int kChunk = 32;    // columns per epilogue chunk
constexpr int kStatCols = 64; // columns per LayerNorm partial; also the row granule in which the AdaLN
                              // shift and scale weight rows are interleaved (64 shift rows | 64 scale rows)
constexpr int kCPad = 16;     // token dim is padded to 16 in Wout^T and the eps partials

enum Epi : int {
  EPI_BIAS_F32 = 0,  // out_f32 = acc0 + bias0                                   (condition projection)
  EPI_SILU_ACT = 1,  // out_act = SiLU(acc0 + bias0)                             (block MLP, first layer)
  EPI_MOD = 2,       // out_act = LN(h)(1 + acc1 + bias1) + acc0 + bias0         (AdaLN modulate)
  EPI_GATE_RES = 3,  // h += (acc1 + bias1) * (acc0 + bias0); LayerNorm partials (second layer + gate)
  EPI_MODF = 4,      // eps partial = Wout^T-tile . [LN(h)(1 + acc1 + bias1) + acc0 + bias0]
  EPI_MODF2 = 5      // the same with 32 output columns: eps_hat | variance parameter (learned-variance heads)
};
constexpr int kCPad2 = 2 * kCPad;   // widest output projection
template <int EPI> __host__ __device__ constexpr bool epi_is_modf() { return EPI == EPI_MODF || EPI == EPI_MODF2; }
// output-projection columns per row (token dim padded to 16, once or twice)
template <int EPI> __host__ __device__ constexpr int epi_out_width() { return EPI == EPI_MODF2 ? kCPad2 : kCPad; }

struct EpiParams {
  int M;                 // valid rows
  int ldo;               // leading dimension (elements) of out / h  (= W or N)
  const float* bias0;    // [N]
  const float* bias1;    // [N]
  float* out_f32;        // EPI_BIAS_F32
  void* out_act;         // EPI_SILU_ACT, EPI_MOD
  float* h;              // EPI_MOD / EPI_MODF (read), EPI_GATE_RES (read-modify-write)
  int nt;                // eps partials per row: N/64 (tensor-core kernel), N/128 (FMA kernel)
  float* stats;          // [M, ldo/64, 2] (mean, M2) per 64-column group of h
  const float* wout_t;   // [N, 16 or 32] fp32, Wout transposed and zero padded (EPI_MODF, EPI_MODF2)
  float* epart;          // [M, nt, 16 or 32] (EPI_MODF, EPI_MODF2)
};

__device__ __forceinline__ float silu_f(float x) { return x / (1.0f + expf(-x)); }
// Fast variant for the tensor-core path (its result is rounded to a 16-bit operand anyway).
__device__ __forceinline__ float silu_fast(float x) {
  // x sigmoid(x) = x/2 (1 + tanh(x/2)): one special-function operation (tanh.approx, relative error about 2^-11,
  // the precision of the 16-bit result) instead of two (exp and reciprocal)
  float t;
  const float hx = 0.5f * x;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(hx));
  return fmaf(hx, t, hx);
}
template <bool FAST> __device__ __forceinline__ float silu_t(float x) { return FAST ? silu_fast(x) : silu_f(x); }

template <typename T> __device__ __forceinline__ T to_act(float v);
template <> __device__ __forceinline__ float to_act<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 to_act<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ __half to_act<__half>(float v) { return __float2half_rn(v); }

template <typename T> __device__ __forceinline__ void store_chunk(T* dst, const float* v);
template <> __device__ __forceinline__ void store_chunk<float>(float* dst, const float* v) {
  float4* d = reinterpret_cast<float4*>(dst);
#pragma unroll
  for (int j = 0; j < 8; ++j) d[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
}
template <> __device__ __forceinline__ void store_chunk<__nv_bfloat16>(__nv_bfloat16* dst, const float* v) {
  uint4* d = reinterpret_cast<uint4*>(dst);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    __nv_bfloat162 p0 = __floats2bfloat162_rn(v[8 * j + 0], v[8 * j + 1]);
    __nv_bfloat162 p1 = __floats2bfloat162_rn(v[8 * j + 2], v[8 * j + 3]);
    __nv_bfloat162 p2 = __floats2bfloat162_rn(v[8 * j + 4], v[8 * j + 5]);
    __nv_bfloat162 p3 = __floats2bfloat162_rn(v[8 * j + 6], v[8 * j + 7]);
    uint4 q;
    q.x = *reinterpret_cast<uint32_t*>(&p0); q.y = *reinterpret_cast<uint32_t*>(&p1);
    q.z = *reinterpret_cast<uint32_t*>(&p2); q.w = *reinterpret_cast<uint32_t*>(&p3);
    d[j] = q;
  }
}

template <> __device__ __forceinline__ void store_chunk<__half>(__half* dst, const float* v) {
  uint4* d = reinterpret_cast<uint4*>(dst);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    __half2 p0 = __floats2half2_rn(v[8 * j + 0], v[8 * j + 1]);
    __half2 p1 = __floats2half2_rn(v[8 * j + 2], v[8 * j + 3]);
    __half2 p2 = __floats2half2_rn(v[8 * j + 4], v[8 * j + 5]);
    __half2 p3 = __floats2half2_rn(v[8 * j + 6], v[8 * j + 7]);
    uint4 q;
    q.x = *reinterpret_cast<uint32_t*>(&p0); q.y = *reinterpret_cast<uint32_t*>(&p1);
    q.z = *reinterpret_cast<uint32_t*>(&p2); q.w = *reinterpret_cast<uint32_t*>(&p3);
    d[j] = q;
  }
}

__device__ __forceinline__ void load_chunk_f32(const float* src, float* v) {
  const float4* s = reinterpret_cast<const float4*>(src);
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    float4 q = s[j];
    v[4 * j] = q.x; v[4 * j + 1] = q.y; v[4 * j + 2] = q.z; v[4 * j + 3] = q.w;
  }
}

// Per-row state carried across the chunks of one tile.
struct RowState {
  float mean, rstd;          // LayerNorm statistics of the row (EPI_MOD, EPI_MODF)
  float eacc[kCPad2];        // output-projection partial sums (EPI_MODF: the first 16; EPI_MODF2: all 32)
  float pm, pm2, pn;         // running (mean, M2, count) of the new h values (EPI_GATE_RES)
};

// Chan et al. merge of two (mean, M2) partials of equal count n (no division): mean = (ma + mb)/2,
// M2 = M2a + M2b + d^2 n/2; b is merged into a.
__device__ __forceinline__ void chan_merge_equal(float& ma, float& m2a, float mb, float m2b, float n) {
  const float d = mb - ma;
  ma = fmaf(d, 0.5f, ma);
  m2a = __fadd_rn(m2a, fmaf(__fmul_rn(d, d), 0.5f * n, m2b));
}

// LayerNorm statistics of row m from its per-64-column (mean, M2) partials.  All partials have the
// same count n = 64, so with G groups  mean = (sum_g mean_g) / G  and
// M2 = sum_g M2_g + n sum_g (mean_g - mean)^2  (Chan et al. for equal counts, all groups at once):
// no chain of dependent divisions.  Sums run in group order, so the result does not depend on which
// CTA computes it.  Up to 24 groups (W <= 1536) are loaded once, as one batch of 16-byte loads.
// CG: read past the L1 cache (the partials were written by other CTAs of the same kernel).
// p: the row's G (mean, M2) pairs, 16-byte aligned.
template <bool CG = false>
__device__ __forceinline__ void row_stats_at(const float4* p, int W, float& mean, float& rstd) {
  const int G = W / kStatCols;   // even: W is a multiple of 128
  constexpr int kB = 12;         // 16-byte loads (two groups each) per batch
  float sum = 0.0f, m2 = 0.0f, q = 0.0f;
  if (G <= 2 * kB) {
    float4 b[kB];
#pragma unroll
    for (int j = 0; j < kB; ++j) b[j] = (2 * j < G) ? (CG ? __ldcg(p + j) : p[j]) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
    for (int j = 0; j < kB; ++j)
      if (2 * j < G) { sum += b[j].x; sum += b[j].z; m2 += b[j].y; m2 += b[j].w; }
    mean = sum / static_cast<float>(G);
#pragma unroll
    for (int j = 0; j < kB; ++j)
      if (2 * j < G) { const float d0 = b[j].x - mean, d1 = b[j].z - mean; q = fmaf(d0, d0, q); q = fmaf(d1, d1, q); }
  } else {
    for (int j = 0; j < G / 2; ++j) { const float4 b = CG ? __ldcg(p + j) : p[j]; sum += b.x; sum += b.z; m2 += b.y; m2 += b.w; }
    mean = sum / static_cast<float>(G);
    for (int j = 0; j < G / 2; ++j) {
      const float4 b = CG ? __ldcg(p + j) : p[j];
      const float d0 = b.x - mean, d1 = b.z - mean;
      q = fmaf(d0, d0, q); q = fmaf(d1, d1, q);
    }
  }
  const float m2t = fmaf(static_cast<float>(kStatCols), q, m2);
  rstd = 1.0f / sqrtf(m2t / static_cast<float>(W) + 1e-6f);
}

template <bool CG = false>
__device__ __forceinline__ void row_stats(const float* stats, int m, int W, float& mean, float& rstd) {
  row_stats_at<CG>(reinterpret_cast<const float4*>(stats) + static_cast<size_t>(m) * (W / kStatCols / 2), W, mean, rstd);
}

template <int EPI>
__device__ __forceinline__ void epi_row_begin(const EpiParams& ep, int m, RowState& rs) {
  if constexpr (EPI == EPI_MOD || epi_is_modf<EPI>()) row_stats<false>(ep.stats, m, ep.ldo, rs.mean, rs.rstd);
  if constexpr (epi_is_modf<EPI>()) {
#pragma unroll
    for (int c = 0; c < epi_out_width<EPI>(); ++c) rs.eacc[c] = 0.0f;
  }
  if constexpr (EPI == EPI_GATE_RES) { rs.pm = 0.0f; rs.pm2 = 0.0f; rs.pn = 0.0f; }
}

template <int EPI> __host__ __device__ constexpr bool epi_reads_h() { return EPI == EPI_MOD || epi_is_modf<EPI>() || EPI == EPI_GATE_RES; }

// Residual update of one 32-column chunk, hv += (a1 + b1) (a0 + b0), and its (mean, M2) partial merged
// into the row state (a thread owns one or two chunks of a 64-column group: the second is merged with
// equal counts).
__device__ __forceinline__ void gate_res_chunk(const float* a0, const float* a1, const float* b0, const float* b1,
                                               float* hv, RowState& rs) {
  float sum = 0.0f;
#pragma unroll
  for (int j = 0; j < kChunk; ++j) {
    const float y = a0[j] + b0[j];
    const float g = a1[j] + b1[j];
    hv[j] = fmaf(g, y, hv[j]);
    sum += hv[j];
  }
  const float mean = sum * (1.0f / kChunk);
  float m2 = 0.0f;
#pragma unroll
  for (int j = 0; j < kChunk; ++j) {
    const float d = hv[j] - mean;
    m2 = fmaf(d, d, m2);
  }
  if (rs.pn <= 0.0f) { rs.pm = mean; rs.pm2 = m2; }
  else chan_merge_equal(rs.pm, rs.pm2, mean, m2, static_cast<float>(kChunk));
  rs.pn += static_cast<float>(kChunk);
}

// AdaLN modulation of one 32-column chunk: a0 <- LN(h)(1 + a1 + b1) + a0 + b0 (a0 = shift, a1 = scale).
__device__ __forceinline__ void modulate_chunk(float* a0, const float* a1, const float* b0, const float* b1,
                                               const float* hv, const RowState& rs) {
#pragma unroll
  for (int j = 0; j < kChunk; ++j) {
    const float shift = a0[j] + b0[j];
    const float scale = a1[j] + b1[j];
    a0[j] = fmaf(__fmul_rn(__fsub_rn(hv[j], rs.mean), rs.rstd), __fadd_rn(1.0f, scale), shift);
  }
}

// Output-projection partial of one chunk: eacc[c] += sum_j a0[j] Wout^T[j][c]  (wout_c: [32][EPW]).
template <int EPW>
__device__ __forceinline__ void outproj_chunk(const float* a0, const float* wout_c, RowState& rs) {
#pragma unroll
  for (int j = 0; j < kChunk; ++j) {
    const float4* w4 = reinterpret_cast<const float4*>(wout_c + j * EPW);
#pragma unroll
    for (int c4 = 0; c4 < EPW / 4; ++c4) {
      const float4 w = w4[c4];
      rs.eacc[4 * c4 + 0] = fmaf(a0[j], w.x, rs.eacc[4 * c4 + 0]);
      rs.eacc[4 * c4 + 1] = fmaf(a0[j], w.y, rs.eacc[4 * c4 + 1]);
      rs.eacc[4 * c4 + 2] = fmaf(a0[j], w.z, rs.eacc[4 * c4 + 2]);
      rs.eacc[4 * c4 + 3] = fmaf(a0[j], w.w, rs.eacc[4 * c4 + 3]);
    }
  }
}

// a0 / a1: accumulator chunk (32 columns) of the first / second accumulator; n0 = first global
// output column of the chunk; b0 / b1: the chunk's 32 biases (shared or global memory); hv: the
// chunk's 32 values of h, already loaded (EPI_MOD, EPI_MODF, EPI_GATE_RES); wout_c: the chunk's
// [32][16 or 32] slice of Wout^T in shared memory (EPI_MODF, EPI_MODF2).
template <int EPI, typename ACT, bool FAST>
__device__ __forceinline__ void epi_chunk(const EpiParams& ep, int m, int n0, float* a0, const float* a1,
                                          const float* b0, const float* b1, float* hv, RowState& rs,
                                          const float* wout_c) {
  const size_t off = static_cast<size_t>(m) * ep.ldo + n0;
  if constexpr (EPI == EPI_BIAS_F32) {
#pragma unroll
    for (int j = 0; j < kChunk; ++j) a0[j] += b0[j];
    store_chunk<float>(ep.out_f32 + off, a0);
  } else if constexpr (EPI == EPI_SILU_ACT) {
#pragma unroll
    for (int j = 0; j < kChunk; ++j) a0[j] = silu_t<FAST>(a0[j] + b0[j]);
    store_chunk<ACT>(reinterpret_cast<ACT*>(ep.out_act) + off, a0);
  } else if constexpr (EPI == EPI_MOD || epi_is_modf<EPI>()) {
    modulate_chunk(a0, a1, b0, b1, hv, rs);
    if constexpr (EPI == EPI_MOD) store_chunk<ACT>(reinterpret_cast<ACT*>(ep.out_act) + off, a0);
    else outproj_chunk<epi_out_width<EPI>()>(a0, wout_c, rs);
  } else if constexpr (EPI == EPI_GATE_RES) {
    gate_res_chunk(a0, a1, b0, b1, hv, rs);
    store_chunk<float>(ep.h + off, hv);
  }
}

// Writes the (mean, M2) partial of one row over 64-column group g.
__device__ __forceinline__ void store_group_stats(const EpiParams& ep, int m, int g, float mean, float m2) {
  reinterpret_cast<float2*>(ep.stats)[static_cast<size_t>(m) * (ep.ldo / kStatCols) + g] = make_float2(mean, m2);
}

template <int EPI>
__device__ __forceinline__ void epi_row_end(const EpiParams& ep, int m, int part, const RowState& rs) {
  if constexpr (epi_is_modf<EPI>()) {
    constexpr int EPW = epi_out_width<EPI>();
    float4* d = reinterpret_cast<float4*>(ep.epart + (static_cast<size_t>(m) * ep.nt + part) * EPW);
#pragma unroll
    for (int c = 0; c < EPW / 4; ++c)
      d[c] = make_float4(rs.eacc[4 * c], rs.eacc[4 * c + 1], rs.eacc[4 * c + 2], rs.eacc[4 * c + 3]);
  }
}

}  // namespace csd
