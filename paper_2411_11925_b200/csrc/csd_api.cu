// C ABI of the continuous speculative decoding hot path (see include/csd.h for the contract).
// Host side: argument checks, weight packing, workspace, launch sequencing.  Every arithmetic step
// runs in the kernels of gemm.cuh / rowops.cuh.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <type_traits>
#include <vector>

#include "../../include/csd.h"
#include "fold.cuh"
#include "gemm.cuh"
#include "gmm.cuh"
#include "rowops.cuh"
#include "smallbatch.cuh"
#include "pchain.cuh"

using namespace csd;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

struct ChainWs {
  void* base = nullptr;
  size_t cap = 0;
  // carved per call
  void *zc, *s, *u, *v;
  float *cz, *te, *h, *stats, *epart, *x;
  void* s2 = nullptr;   // s of even steps (s of odd steps: s)
  void* ap = nullptr;   // a' = h (1 + scale) of the folded blocks
  float* hid = nullptr; // hidden layer of the timestep embedding [T, W]
  bool owned = true;    // false: base is memory the library did not allocate and must never free or grow
};

constexpr int kMaxDevices = 64;   // device ordinals the per-device tables below cover

struct ProfRec { cudaEvent_t a, b; int cls; double flops; };

struct HostIo {  // device mirrors for csd_round_host
  void* base = nullptr;
  size_t cap = 0;
};

}  // namespace

struct csd_ctx {
  int device = 0;
  int num_sms = 148;
  cudaStream_t stream = nullptr;
  cudaStream_t side[2] = {nullptr, nullptr};
  cudaEvent_t ev_fork = nullptr, ev_done[2] = {nullptr, nullptr};
  int* d_err = nullptr;
  int64_t launches = 0;
  int chain_mode = CSD_CHAIN_LAYERS;   // csd_set_chain_mode
  EncodeTiledFn encode = nullptr;
  ChainWs ws[3];   // draft chain, target chain, static-scratch calls
  HostIo io;
  HostIo un;       // csd_verify_unaligned: per-row noise terms
  HostIo bn;       // csd_bonus_token: samples of every sequence before the selection
  HostIo sp;       // csd_verify_single_path: schedule constants, mu^p of one pass, running log-ratio
  HostIo pc[3];    // persistent chain kernel (per chain slot): s of all steps, a', v, partials, counters, schedule
  HostIo sb[2];    // small-batch chain kernel (per chain slot): s of all steps, early products, a', v, counters, schedule
  char err[512] = {0};
  // optional per-launch timing (csd_profile)
  bool prof_on = false;
  std::vector<ProfRec> prof;
  std::vector<cudaEvent_t> ev_pool;
  size_t ev_used = 0;
};

struct csd_head {
  csd_ctx* ctx = nullptr;
  csd_head_desc d{};
  void* wblob = nullptr;   // GEMM weights (bf16 or fp32)
  float* fblob = nullptr;  // fp32 side parameters
  size_t esz = 4;
  // GEMM weights
  void* Wz = nullptr;
  std::vector<void*> Wss, Wg, W1, W2;
  void* Wfss = nullptr;
  // fp32 parameters
  float *bz, *Wt1, *bt1, *Wt2, *bt2, *win, *bin, *bfsh, *bfsc, *wout_t, *bout;
  std::vector<float*> bsh, bsc, bg, b1, b2;
  // tensor maps of the weights (16-bit heads), one set per output-tile width: [0] 64, [1] 128 columns
  struct TmSet {
    CUtensorMap Wz{}, Wfss{};
    std::vector<CUtensorMap> Wss, Wg, W1, W2;
  } tm[2];
  std::vector<CUtensorMap> W1_wide;
  // folded blocks (fold.cuh): packed [Wg_k | Wscale_{k+1}] (k < L-1) and [W1_k Wscale_k | W1_k Wshift_k] (k >= 1),
  // 256-row boxes; c1_k = W1_k (1 + bscale_k), c2_k = W1_k bshift_k + b1_k
  void* xblob = nullptr;
  std::vector<CUtensorMap> Wgs, Wf;
  std::vector<CUtensorMap> Wgs_half, Wf_half;   // the same matrices in 128-row boxes: what one CTA of a pair loads
  std::vector<float*> c1, c2;   // first MLP layer with 256-row boxes (W a multiple of 256)
  // small-batch chain kernel (smallbatch.cuh): usable for this head; device tables (tensor maps of W1_k, W2_k, then of
  // the matrices multiplied by s: per block Wf_k, Wg_k, Wss_k, then Wfss, all in 128-row boxes; early tiles; biases)
  bool sb_ready = false;
  // persistent chain kernel (pchain.cuh): per phase the early and the dependent weight maps; per phase three bias rows
  bool pc_ready = false;
  CUtensorMap* d_pc_maps = nullptr;
  const float** d_pc_bias = nullptr;
  int sb_ntasks = 0;
  CUtensorMap* d_sb_maps = nullptr;
  SbTask* d_sb_tasks = nullptr;
  const float** d_sb_bias = nullptr;
};

namespace {

int fail(csd_ctx* ctx, int code, const char* fmt, ...) {
  if (ctx) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
    va_end(ap);
  }
  return code;
}

#define CSD_CUDA(ctx, call)                                                                          \
  do {                                                                                               \
    cudaError_t e_ = (call);                                                                         \
    if (e_ != cudaSuccess)                                                                           \
      return fail(ctx, CSD_ERR_CUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_), __FILE__, \
                  __LINE__);                                                                         \
  } while (0)

// Makes the context's device current for the duration of a call and puts the caller's device back afterwards.
struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { prev = -1; cudaGetLastError(); }
    if (prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
  DeviceGuard(const DeviceGuard&) = delete;
  DeviceGuard& operator=(const DeviceGuard&) = delete;
};
#define CSD_DEVICE(ctx)                                                                              \
  DeviceGuard device_guard_((ctx)->device);                                                          \
  if (!device_guard_.ok) return fail(ctx, CSD_ERR_CUDA, "cannot make device %d current", (ctx)->device)

cudaEvent_t prof_event(csd_ctx* ctx) {
  if (ctx->ev_used == ctx->ev_pool.size()) {
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
    ctx->ev_pool.push_back(e);
  }
  return ctx->ev_pool[ctx->ev_used++];
}
// Brackets one launch with events on its own stream when profiling is on.
struct ProfScope {
  csd_ctx* ctx; cudaStream_t st; cudaEvent_t a = nullptr, b = nullptr; int cls; double flops;
  ProfScope(csd_ctx* c, cudaStream_t s, int cls_, double fl) : ctx(c), st(s), cls(cls_), flops(fl) {
    if (ctx->prof_on && (a = prof_event(ctx)) && (b = prof_event(ctx))) cudaEventRecord(a, st);
  }
  ~ProfScope() {
    if (a && b) { cudaEventRecord(b, st); ctx->prof.push_back({a, b, cls, flops}); }
  }
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

uint16_t f32_to_bf16_bits(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return static_cast<uint16_t>((u >> 16) | 0x40);  // NaN
  const uint32_t bias = ((u >> 16) & 1u) + 0x7fffu;
  return static_cast<uint16_t>((u + bias) >> 16);
}

int make_tmap(csd_ctx* ctx, CUtensorMap* m, int dtype, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld,
              uint32_t box_rows) {
  const cuuint64_t gdim[2] = {cols, rows};
  const cuuint64_t gstride[1] = {ld * 2};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBlockK), box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = ctx->encode(m, dtype == CSD_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box,
                                 estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(ctx, CSD_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return CSD_OK;
}

// fp32 [rows, cols] matrix read in boxes of 32 floats (128 bytes, swizzled) x 128 rows.
int make_tmap_f32(csd_ctx* ctx, CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols) {
  const cuuint64_t gdim[2] = {cols, rows};
  const cuuint64_t gstride[1] = {cols * 4};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(kChunk), static_cast<cuuint32_t>(kTileM)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = ctx->encode(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(ptr), gdim, gstride, box, estr,
                                 CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(ctx, CSD_ERR_CUDA, "cuTensorMapEncodeTiled (fp32) failed with code %d", (int)r);
  return CSD_OK;
}

// Byte offsets of a chain's intermediates inside its workspace (each piece rounded up to 1 KiB) and their total.
// The one place that knows the layout: the growable workspaces and the fixed static scratch both use it.
struct WsLayout {
  size_t zc, s, u, v, cz, te, h, stats, epart, x, ap, hid, s2, total;
};

WsLayout ws_layout(const csd_head_desc& d, int Rh, int R, int T) {
  const size_t asz = d.dtype == CSD_F32 ? 4 : 2;
  const size_t W = d.W, rh = static_cast<size_t>(Rh);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
  WsLayout l{};
  l.zc = take(rh * d.Dz * asz);
  l.s = take(rh * W * asz); l.u = take(rh * W * asz); l.v = take(rh * W * asz);
  l.cz = take(rh * W * 4); l.te = take(static_cast<size_t>(T) * W * 4); l.h = take(rh * W * 4);
  l.stats = take(rh * (W / kStatCols) * 8);
  l.epart = take(rh * (W / kStatCols) * (d.var_out ? kCPad2 : kCPad) * 4);   // room for 64-wide tiles
  l.x = take(static_cast<size_t>(R) * kCPad * 4);
  l.ap = take(d.dtype == CSD_F32 ? 0 : rh * W * asz);
  l.hid = take(static_cast<size_t>(T) * W * 4);
  l.s2 = take(rh * W * asz);
  l.total = off;
  return l;
}

int ensure_ws(csd_ctx* ctx, ChainWs& ws, const csd_head_desc& d, int Rh, int R, int T) {
  const WsLayout l = ws_layout(d, Rh, R, T);
  if (l.total > ws.cap) {
    if (!ws.owned) return fail(ctx, CSD_ERR_WORKSPACE, "the fixed scratch holds %zu bytes, this call needs %zu", ws.cap, l.total);
    CSD_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    for (int i = 0; i < 2; ++i) CSD_CUDA(ctx, cudaStreamSynchronize(ctx->side[i]));
    if (ws.base) CSD_CUDA(ctx, cudaFree(ws.base));
    ws.base = nullptr;
    ws.cap = 0;
    if (cudaMalloc(&ws.base, l.total) != cudaSuccess) {
      cudaGetLastError();
      return fail(ctx, CSD_ERR_WORKSPACE, "cannot allocate %zu bytes of workspace", l.total);
    }
    ws.cap = l.total;
  }
  char* b = static_cast<char*>(ws.base);
  ws.zc = b + l.zc; ws.s = b + l.s; ws.u = b + l.u; ws.v = b + l.v;
  ws.cz = reinterpret_cast<float*>(b + l.cz); ws.te = reinterpret_cast<float*>(b + l.te);
  ws.h = reinterpret_cast<float*>(b + l.h); ws.stats = reinterpret_cast<float*>(b + l.stats);
  ws.epart = reinterpret_cast<float*>(b + l.epart); ws.x = reinterpret_cast<float*>(b + l.x);
  ws.ap = b + l.ap; ws.hid = reinterpret_cast<float*>(b + l.hid);
  ws.s2 = b + l.s2;
  return CSD_OK;
}

template <int EPI, int NSEG, int NMUL, int TN, typename ACT, bool PAIR>
int launch_tc_t(csd_ctx* ctx, cudaStream_t st, const CUtensorMap& a0, const CUtensorMap& b0, const CUtensorMap& a1,
                const CUtensorMap& b1, const CUtensorMap& th, int K0, int K1, int dep_k, int N, const EpiParams& ep,
                const CUtensorMap* tout = nullptr) {
  constexpr int MMA_N = NMUL * TN;
  auto kern = gemm_tc_kernel<EPI, ACT, NSEG, MMA_N, TN, std::is_same<ACT, __half>::value ? 0 : 1, PAIR>;
  static bool attr_done[kMaxDevices] = {};   // function attributes are per device
  constexpr int smem = TcCfg<EPI, MMA_N, TN, PAIR>::kSmemBytes;
  if (!attr_done[ctx->device]) {
    CSD_CUDA(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    attr_done[ctx->device] = true;
  }
  // Work units: output tiles, or pair tiles (two row tiles) for CTA pairs.  Persistent: at most one CTA per SM.
  const int tiles_n = N / TN, row_tiles = (ep.M + kTileM - 1) / kTileM;
  const int units = tiles_n * (PAIR ? (row_tiles + 1) / 2 : row_tiles);
  const int max_units = PAIR ? ctx->num_sms / 2 : ctx->num_sms;
  dim3 grid((units < max_units ? units : max_units) * (PAIR ? 2 : 1));
  ProfScope ps(ctx, st, EPI == EPI_MODF2 ? EPI_MODF : EPI, 2.0 * ep.M * static_cast<double>(N) * (K0 + K1) * NMUL);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = dim3(TcWarps<EPI, TN>::kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (PAIR) {
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = 2; at[na].val.clusterDim.y = 1; at[na].val.clusterDim.z = 1;
    ++na;
  }
  if (!ctx->prof_on) {   // event pairs between launches defeat the overlap anyway
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = at; cfg.numAttrs = na;
  EpiParams e = ep;
  e.nt = N / kStatCols;   // eps partials are per 64-column group for both tile widths
  CSD_CUDA(ctx, cudaLaunchKernelEx(&cfg, kern, a0, b0, a1, b1, th, tout ? *tout : th, K0 / kBlockK, K1 / kBlockK, dep_k / kBlockK, tiles_n, units, e,
                                   ctx->d_err));
  ctx->launches++;
  return CSD_OK;
}

// NMUL = 2: B holds the interleaved AdaLN shift | scale rows (two accumulator columns per output column).
// tn: output columns per CTA, 64 or 128; pair: two CTAs share each MMA (needs tn = 128; the B tensor maps
// b0 / b1 then have half-height boxes).  dep_k: first K index (over both segments) whose A operand is
// written by the preceding kernel.
template <int EPI, int NSEG, int NMUL>
int launch_tc(csd_ctx* ctx, int dtype, int tn, bool pair, cudaStream_t st, const CUtensorMap& a0, const CUtensorMap& b0,
              const CUtensorMap& a1, const CUtensorMap& b1, const CUtensorMap& th, int K0, int K1, int dep_k,
              int N, const EpiParams& ep, const CUtensorMap* tout = nullptr) {
  if (dtype == CSD_F16) {
    if (tn == 64) return launch_tc_t<EPI, NSEG, NMUL, 64, __half, false>(ctx, st, a0, b0, a1, b1, th, K0, K1, dep_k, N, ep, tout);
    if (pair) return launch_tc_t<EPI, NSEG, NMUL, 128, __half, true>(ctx, st, a0, b0, a1, b1, th, K0, K1, dep_k, N, ep, tout);
    return launch_tc_t<EPI, NSEG, NMUL, 128, __half, false>(ctx, st, a0, b0, a1, b1, th, K0, K1, dep_k, N, ep, tout);
  }
  if (tn == 64) return launch_tc_t<EPI, NSEG, NMUL, 64, __nv_bfloat16, false>(ctx, st, a0, b0, a1, b1, th, K0, K1, dep_k, N, ep, tout);
  if (pair) return launch_tc_t<EPI, NSEG, NMUL, 128, __nv_bfloat16, true>(ctx, st, a0, b0, a1, b1, th, K0, K1, dep_k, N, ep, tout);
  return launch_tc_t<EPI, NSEG, NMUL, 128, __nv_bfloat16, false>(ctx, st, a0, b0, a1, b1, th, K0, K1, dep_k, N, ep, tout);
}

template <int EPI, int NSEG, int MMA_N>
int launch_simt(csd_ctx* ctx, cudaStream_t st, const float* A0, int lda0, const float* B0, int K0, const float* A1,
                int lda1, const float* B1, int K1, int N, const EpiParams& ep) {
  dim3 grid(N / kTileN, (ep.M + kSimtRows - 1) / kSimtRows);
  ProfScope ps(ctx, st, EPI == EPI_MODF2 ? EPI_MODF : EPI, 2.0 * ep.M * static_cast<double>(N) * (K0 + K1) * ((NSEG == 1 && MMA_N == 256) ? 2.0 : 1.0));
  EpiParams e = ep;
  e.nt = N / kTileN;
  gemm_simt_kernel<EPI, NSEG, MMA_N><<<grid, 128, 0, st>>>(A0, lda0, B0, K0, K0, A1, lda1, B1, K1, K1, e);
  ctx->launches++;
  CSD_CUDA(ctx, cudaGetLastError());
  return CSD_OK;
}

int check_sched(csd_ctx* ctx, const csd_schedule* s, bool full) {
  if (!s) return fail(ctx, CSD_ERR_INVALID_ARG, "schedule is null");
  if (s->T < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "schedule T = %d must be >= 1", s->T);
  if (!s->sigma) return fail(ctx, CSD_ERR_INVALID_ARG, "schedule sigma is null");
  if (full && (!s->a || !s->b || !s->tfeat)) return fail(ctx, CSD_ERR_INVALID_ARG, "schedule a/b/tfeat is null");
  for (int t = 0; t < s->T; ++t)
    if (!(s->sigma[t] > 0.0f)) return fail(ctx, CSD_ERR_INVALID_ARG, "schedule sigma[%d] must be > 0", t);
  return CSD_OK;
}

// Chains whose layers are one wave of tiles run as one persistent kernel (pchain.cuh) where it applies.
#ifndef CSD_PERSISTENT_CHAINS
#define CSD_PERSISTENT_CHAINS 1
#endif
constexpr bool kPersistentChains = CSD_PERSISTENT_CHAINS != 0;

// Folded blocks run as CTA pairs when a layer's row tiles pair up.
#ifndef CSD_FOLD_PAIRS
#define CSD_FOLD_PAIRS 1
#endif
constexpr bool kFoldPairs = CSD_FOLD_PAIRS != 0;

// Shared-memory opt-in of the folded block kernels, once per device and operand type.
bool fold_kernels_ready(const csd_ctx* ctx, const csd_head_desc& d) {
  static int known[kMaxDevices][2] = {};
  int& k = known[ctx->device][d.dtype == CSD_F16 ? 0 : 1];
  if (k == 0) {
    bool ok = true;
    if (d.dtype == CSD_F16) {
      ok = ok && cudaFuncSetAttribute(fold_kernel<__half, 0, FOLD_W1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FoldCfg<FOLD_W1>::kSmemBytes) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(fold_kernel<__half, 0, FOLD_GATE, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FoldCfg<FOLD_GATE>::kSmemBytes) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(fold_kernel<__half, 0, FOLD_W1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FoldCfg<FOLD_W1>::kSmemBytes) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(fold_kernel<__half, 0, FOLD_GATE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FoldCfg<FOLD_GATE>::kSmemBytes) == cudaSuccess;
    } else {
      ok = ok && cudaFuncSetAttribute(fold_kernel<__nv_bfloat16, 1, FOLD_W1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FoldCfg<FOLD_W1>::kSmemBytes) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(fold_kernel<__nv_bfloat16, 1, FOLD_GATE, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FoldCfg<FOLD_GATE>::kSmemBytes) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(fold_kernel<__nv_bfloat16, 1, FOLD_W1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FoldCfg<FOLD_W1>::kSmemBytes) == cudaSuccess;
      ok = ok && cudaFuncSetAttribute(fold_kernel<__nv_bfloat16, 1, FOLD_GATE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FoldCfg<FOLD_GATE>::kSmemBytes) == cudaSuccess;
    }
    cudaGetLastError();
    k = ok ? 1 : -1;
  }
  return k == 1;
}

int ensure_side(csd_ctx* ctx, HostIo& io, size_t need, const char* what);

// Shared-memory opt-in of the persistent chain kernel, once per device and operand type.
bool pchain_kernel_ready(const csd_ctx* ctx, int dtype) {
  static int known[kMaxDevices][2] = {};
  int& k = known[ctx->device][dtype == CSD_F16 ? 0 : 1];
  if (k == 0) {
    const bool ok = dtype == CSD_F16
        ? cudaFuncSetAttribute(pchain_kernel<__half, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPcSmemBytes) == cudaSuccess
        : cudaFuncSetAttribute(pchain_kernel<__nv_bfloat16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPcSmemBytes) == cudaSuccess;
    cudaGetLastError();
    k = ok ? 1 : -1;
  }
  return k == 1;
}

// Whether the small-batch chain kernel can run on this device: its clusters of 8 CTAs (one per SM, ~213 KB of
// shared memory each) must all be resident at once.  Returns the number of clusters the GPU holds (0: unusable).
template <typename ACT, int FMT>
int sb_clusters_of(csd_ctx* ctx) {
  static int known[kMaxDevices] = {};   // 0 unknown, > 0 clusters, -1 unusable
  int& k = known[ctx->device];
  if (k == 0) {
    k = -1;
    auto kern = sb_chain_kernel<ACT, FMT>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSbSmemBytes) == cudaSuccess &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 0) == cudaSuccess) {
      cudaLaunchConfig_t lc{};
      lc.gridDim = dim3(kSbCluster); lc.blockDim = dim3(kSbThreads); lc.dynamicSmemBytes = kSbSmemBytes;
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = kSbCluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      lc.attrs = at; lc.numAttrs = 1;
      int ncl = 0;
      if (cudaOccupancyMaxActiveClusters(&ncl, kern, &lc) == cudaSuccess && ncl >= 1) k = ncl;
    }
    cudaGetLastError();
  }
  return k > 0 ? k : 0;
}

// One head's denoising chain for R token rows on stream `st` with workspace slot `slot`:
// begin() enqueues the per-call work (timestep embedding, condition projection, first boundary
// kernel), step(t) enqueues the kernels of step t.  Two chains can be interleaved launch by launch.
struct Chain {
  csd_ctx* ctx; int slot; cudaStream_t st; const csd_head* hd; const csd_schedule* sc;
  int R, cfg; float cfg_scale; const float *z, *x_T, *eps; int sample_last; float *x0, *mu1, *x1;
  int chains = 1;   // chains that run concurrently with this one (itself included)
  int Rh = 0, W = 0, L = 0, T = 0, tn = kTileN;
  bool sbk = false;       // the whole chain runs in the small-batch kernel (smallbatch.cuh)
  bool pck = false;       // the whole chain runs in the persistent chain kernel (pchain.cuh)
  bool fold = false;      // blocks 1.. run as two kernels (fold.cuh) instead of three
  CUtensorMap tm_ap{};
  bool mod64 = false;     // modulate kernels in 64-wide tiles although the others use 128
  bool w1_wide = false;   // first MLP layer in 128 x 256 tiles (MMA N = 256)
  bool tc = false, pair = false;
  // s is double-buffered by step parity (index t & 1): the boundary kernel that ends step t writes s of step t - 2,
  // so no product of s ever waits for the kernel right before it
  CUtensorMap tm_z{}, tm_sb[2]{}, tm_u{}, tm_v{}, tm_h{};
  void* sbuf[2] = {nullptr, nullptr};
  int cur_t = 0;
  EpiParams ep{};
  StepParams sp{};
  // trajectory recording (csd_draft_denoise_traj): [T + 1, R, C] states and [T, R, C] means, or null
  float *traj_x = nullptr, *traj_mu = nullptr;
  // learned-variance heads: host arrays [T] of the log-variance bounds, outputs lv1 [R, C] and half_logdet [R]
  const float *lv_min = nullptr, *lv_max = nullptr;
  float *lv1 = nullptr, *half_logdet = nullptr;
  // batched evaluation on a given trajectory (csd_verify_single_path): R = batch_steps * batch_Rin token rows,
  // one pass of the layers; slot batch_j0 of batch_traj is the first step of the pass
  int batch_Rin = 0, batch_j0 = 0, Ts = 0;
  int ws_steps = 0;          // steps the workspace is carved for (the same for every pass of a call, so that the
  bool batch_reuse = false;  // timestep embedding and the condition projection of the first pass stay where they are)
  const float *batch_traj = nullptr, *batch_sched = nullptr;
  float* batch_mu = nullptr;

  template <typename ACT>
  int launch_step_t(cudaLaunchConfig_t& cfg, bool rb4, int mode) {
    if (lv_min) CSD_CUDA(ctx, cudaLaunchKernelEx(&cfg, rb4 ? step_kernel<ACT, 4, false, true> : step_kernel<ACT, 1, false, true>, sp, mode));
    else if (traj_x) CSD_CUDA(ctx, cudaLaunchKernelEx(&cfg, rb4 ? step_kernel<ACT, 4, true> : step_kernel<ACT, 1, true>, sp, mode));
    else CSD_CUDA(ctx, cudaLaunchKernelEx(&cfg, rb4 ? step_kernel<ACT, 4> : step_kernel<ACT, 1>, sp, mode));
    return CSD_OK;
  }

  // kind 0: prepare the pass (h, LayerNorm partials, s); kind 1: finish it (eps_hat, guidance, mu^p)
  int launch_batch(int kind) {
    const csd_head_desc& d = hd->d;
    ChainWs& ws = ctx->ws[slot];
    BatchParams b{};
    b.Rin = batch_Rin; b.Rtok = R; b.cfg = cfg; b.C = d.C; b.W = W; b.NT = tc ? W / kStatCols : W / kTileN;
    b.T = Ts; b.j0 = batch_j0; b.cfg_scale = cfg_scale; b.sched = batch_sched; b.traj_x = batch_traj;
    b.win = hd->win; b.bin = hd->bin; b.cz = ws.cz; b.te = ws.te; b.h = ws.h; b.stats = ws.stats; b.s = ws.s;
    b.epart = ws.epart; b.bout = hd->bout; b.mu_p = batch_mu; b.status = ctx->d_err + 1;
    ProfScope ps(ctx, st, 5, 2.0 * Rh * static_cast<double>(W) * d.C);
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(kind == 0 ? (R + 3) / 4 : (R + 15) / 16); lc.blockDim = dim3(256); lc.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at; lc.numAttrs = (ctx->prof_on || !tc) ? 0 : 1;
    if (kind == 1) CSD_CUDA(ctx, cudaLaunchKernelEx(&lc, batch_finish_kernel, b));
    else if (d.dtype == CSD_F16) CSD_CUDA(ctx, cudaLaunchKernelEx(&lc, batch_prepare_kernel<__half>, b));
    else if (d.dtype == CSD_BF16) CSD_CUDA(ctx, cudaLaunchKernelEx(&lc, batch_prepare_kernel<__nv_bfloat16>, b));
    else CSD_CUDA(ctx, cudaLaunchKernelEx(&lc, batch_prepare_kernel<float>, b));
    ctx->launches++;
    CSD_CUDA(ctx, cudaGetLastError());
    return CSD_OK;
  }

  int launch_step(int mode) {
    const csd_head_desc& d = hd->d;
    ProfScope ps(ctx, st, 5, 2.0 * Rh * static_cast<double>(W) * d.C);
    cudaLaunchConfig_t cfg{};
    // four token rows per block once that still leaves every SM several blocks (the choice does not change a bit)
    const bool rb4 = R >= 8 * ctx->num_sms;
    cfg.gridDim = dim3(rb4 ? (R + 3) / 4 : R); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = 0; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = (ctx->prof_on || !tc) ? 0 : 1;
    int rc;
    if (d.dtype == CSD_F16) rc = launch_step_t<__half>(cfg, rb4, mode);
    else if (d.dtype == CSD_BF16) rc = launch_step_t<__nv_bfloat16>(cfg, rb4, mode);
    else rc = launch_step_t<float>(cfg, rb4, mode);
    if (rc) return rc;
    ctx->launches++;
    CSD_CUDA(ctx, cudaGetLastError());
    return CSD_OK;
  }

  int begin() {
    const csd_head_desc& d = hd->d;
    Rh = R * (cfg ? 2 : 1); W = d.W; L = d.L; Ts = sc->T;
    T = batch_Rin ? 1 : Ts;   // a batched pass runs the layers once
    tc = d.dtype != CSD_F32;
    // 64-wide output tiles when 128-wide ones (of all chains running side by side) would occupy at most a
    // quarter of the SMs: a kernel and the early part of its successor should both find free SMs
    tn = (tc && chains * (W / kTileN) * ((Rh + kTileM - 1) / kTileM) <= ctx->num_sms / 4) ? 64 : kTileN;
    // CTA pairs (two row tiles per MMA, half of each weight tile per CTA) need 128-wide tiles; they are
    // used once a kernel has at least two waves of tiles, where L2-to-SM bandwidth is the limit (measured:
    // a few per cent faster at 384 tiles, slower at 64 and 256)
    pair = tc && tn == kTileN && (W / kTileN) * ((Rh + kTileM - 1) / kTileM) >= 2 * ctx->num_sms;
    // First MLP layer: 256-wide MMAs keep the tensor pipe busier per issued instruction (measured about 660 clk
    // per 64-deep k-block and tile against 415 for two 128-wide tiles' worth), but halve the tile count; taken when
    // that does not cost a wave.
    {
      const int row_tiles = (Rh + kTileM - 1) / kTileM, t128 = (W / kTileN) * row_tiles, t256 = (W / 256) * row_tiles;
      const int waves128 = (t128 + ctx->num_sms - 1) / ctx->num_sms, waves256 = (t256 + ctx->num_sms - 1) / ctx->num_sms;
      w1_wide = tc && !pair && tn == kTileN && W % 256 == 0 && waves256 * 664 < waves128 * 415;
    }
    // The modulate kernels' products never wait for the preceding kernel, only their epilogues do: with 64-wide
    // tiles the epilogue a thread runs is half as long.  Taken for a chain that has the GPU to itself and whose
    // 64-wide tiles fit one wave (measured: draft chain of mar256 10.4 -> 9.8 ms, target chain 18.2 -> 17.7 ms;
    // with two chains side by side the extra CTAs cost more than they save).
    mod64 = tc && chains == 1 && tn == kTileN && !pair && 2 * (W / kTileN) * ((Rh + kTileM - 1) / kTileM) <= ctx->num_sms;
    // Folded blocks: one 128-wide tile per CTA, and their early products want idle SMs to overlap the preceding
    // kernel: taken when the layer's tiles fill between an eighth and half of the SMs (measured slower on tiny grids,
    // which run 64-wide tiles, and on a full wave)
    // (the rule looks at this chain alone, so that csd_round and the three separate calls take the same path).
    {
      const int t128 = (W / kTileN) * ((Rh + kTileM - 1) / kTileM);
      fold = tc && (ctx->chain_mode == CSD_CHAIN_LAYERS || ctx->chain_mode == CSD_CHAIN_LAYER_KERNELS) && !pair && L >= 2 && !hd->Wf.empty() &&
             8 * t128 > ctx->num_sms && 2 * t128 <= ctx->num_sms && fold_kernels_ready(ctx, d);
    }
    // Few rows: one persistent kernel for the whole chain (opt-in per context).  It needs the GPU to itself, so a
    // round that uses it runs its two chains one after the other (chains == 1 here).
    sbk = tc && ctx->chain_mode == CSD_CHAIN_SMALL_BATCH && Rh <= kSbRows && hd->sb_ready && chains == 1 && slot != 2 &&
          !traj_x && !batch_Rin && !lv_min && !ctx->prof_on &&
          (d.dtype == CSD_F16 ? sb_clusters_of<__half, 0>(ctx) : sb_clusters_of<__nv_bfloat16, 1>(ctx)) > kSbRows / kSbGroup;
    if (sbk) { fold = false; pair = false; }
    // One wave of 128 x 128 tiles per layer and W = 1024: one persistent kernel per chain (pchain.cuh).  Row blocks are
    // paired: an odd number is rounded up with a block of rows that belong to no token.
    {
      const int row_tiles = (Rh + kTileM - 1) / kTileM, nb = cfg ? (R + 63) / 64 : (R + 127) / 128;
      const int t128 = (W / kTileN) * row_tiles;
      pck = kPersistentChains && tc && ctx->chain_mode == CSD_CHAIN_LAYERS && !pair && !sbk && slot != 2 && hd->pc_ready &&
            8 * t128 > ctx->num_sms && 2 * t128 <= ctx->num_sms && W / kTileN == kPcColTiles && row_tiles == nb &&
            !batch_Rin && !lv_min && !ctx->prof_on && d.C <= kCPad && pchain_kernel_ready(ctx, d.dtype);
      if (pck) { fold = false; pair = false; }
    }
    ChainWs& ws = ctx->ws[slot];
    int rc = batch_Rin ? ensure_ws(ctx, ws, d, ws_steps * batch_Rin * (cfg ? 2 : 1), ws_steps * batch_Rin, Ts)
                       : ensure_ws(ctx, ws, d, Rh, R, Ts);
    if (rc) return rc;
    if (!batch_reuse) {
      const dim3 grid((W + 31) / 32, (Ts + 31) / 32);
      small_gemm_nt_kernel<true><<<grid, 256, 0, st>>>(sc->tfeat, hd->Wt1, hd->bt1, ws.hid, Ts, W, d.F);
      small_gemm_nt_kernel<false><<<grid, 256, 0, st>>>(ws.hid, hd->Wt2, hd->bt2, ws.te, Ts, W, W);
      ctx->launches += 2;
    }
    CSD_CUDA(ctx, cudaGetLastError());
    ep.M = Rh; ep.ldo = W;
    // rows of z: one per head row, or one per row of a step when the steps of a trajectory are batched
    const int Rz = batch_Rin ? batch_Rin * (cfg ? 2 : 1) : Rh;
    if (tc) {
      if (!batch_reuse) {
        const size_t nz = static_cast<size_t>(Rz) * d.Dz;
        const unsigned nblk = static_cast<unsigned>((nz + 255) / 256);
        if (d.dtype == CSD_F16) convert_act_kernel<__half><<<nblk, 256, 0, st>>>(z, static_cast<__half*>(ws.zc), nz);
        else convert_act_kernel<__nv_bfloat16><<<nblk, 256, 0, st>>>(z, static_cast<__nv_bfloat16*>(ws.zc), nz);
        ctx->launches++;
      }
      if ((rc = make_tmap(ctx, &tm_z, d.dtype, ws.zc, Rz, d.Dz, d.Dz, kTileM))) return rc;
      if ((rc = make_tmap(ctx, &tm_sb[1], d.dtype, ws.s, Rh, W, W, kTileM))) return rc;
      if ((rc = make_tmap(ctx, &tm_sb[0], d.dtype, ws.s2, Rh, W, W, kTileM))) return rc;
      if ((rc = make_tmap(ctx, &tm_u, d.dtype, ws.u, Rh, W, W, kTileM))) return rc;
      if ((rc = make_tmap(ctx, &tm_v, d.dtype, ws.v, Rh, W, W, kTileM))) return rc;
      if ((rc = make_tmap_f32(ctx, &tm_h, ws.h, Rh, W))) return rc;
      if ((rc = make_tmap(ctx, &tm_ap, d.dtype, ws.ap, Rh, W, W, kTileM))) return rc;
    }
    // cz = z Wz^T + bz
    const csd_head::TmSet& tmw = hd->tm[(tn == 64 || pair) ? 0 : 1];   // pairs load half of each B tile per CTA
    EpiParams e = ep;
    e.M = Rz;
    e.bias0 = hd->bz; e.out_f32 = ws.cz;
    if (batch_reuse) rc = CSD_OK;
    else if (tc) rc = launch_tc<EPI_BIAS_F32, 1, 1>(ctx, d.dtype, tn, pair, st, tm_z, tmw.Wz, tm_z, tmw.Wz, tm_h, d.Dz, 0, 0, W, e);
    else rc = launch_simt<EPI_BIAS_F32, 1, 128>(ctx, st, z, d.Dz, static_cast<const float*>(hd->Wz), d.Dz, nullptr, 0,
                                                nullptr, 0, W, e);
    if (rc) return rc;
    sbuf[0] = ws.s2; sbuf[1] = ws.s;
    if (sbk) return launch_small_batch();
    if (pck) return launch_pchain();
    if (batch_Rin) return launch_batch(0);   // a pass has one step (t = 1): its s is sbuf[1]
    sp.traj_x = traj_x; sp.traj_mu = nullptr; sp.status = ctx->d_err + 1;
    sp.lv1 = lv1; sp.half_logdet = half_logdet; sp.lv_min = 0.0f; sp.lv_max = 0.0f;
    sp.R = R; sp.cfg = cfg; sp.C = d.C; sp.W = W; sp.NT = tc ? W / kStatCols : W / kTileN; sp.cfg_scale = cfg_scale;
    sp.sample_last = sample_last; sp.epart = ws.epart; sp.bout = hd->bout; sp.x_src = x_T; sp.x = ws.x;
    sp.x0 = x0; sp.mu1 = mu1; sp.x1 = x1; sp.win = hd->win; sp.bin = hd->bin; sp.cz = ws.cz; sp.h = ws.h;
    sp.stats = ws.stats; sp.s = sbuf[T & 1];
    sp.te_next = ws.te + static_cast<size_t>(T - 1) * W;
    sp.s_b = T >= 2 ? sbuf[(T - 1) & 1] : nullptr;   // the first boundary also prepares s of step T - 1
    sp.te_b = T >= 2 ? ws.te + static_cast<size_t>(T - 2) * W : nullptr;
    sp.eps_t = eps;
    return launch_step(STEP_INIT);
  }

  int launch_fold(int kind, int k) {
    const csd_head_desc& d = hd->d;
    ChainWs& ws = ctx->ws[slot];
    FoldParams p{};
    p.M = Rh; p.W = W; p.err = ctx->d_err;
    const int tiles_n = W / kTileN, row_tiles = (Rh + kTileM - 1) / kTileM;
    // CTA pairs (two row tiles per MMA) whenever the row tiles pair up
    const bool fp = kFoldPairs && row_tiles % 2 == 0;
    const CUtensorMap *tp, *ta, *tw, *tout;
    if (kind == FOLD_W1) {
      p.c0 = hd->c1[k]; p.c1 = hd->c2[k]; p.c2 = nullptr; p.stats_in = ws.stats; p.out = ws.v;
      tp = fp ? &hd->Wf_half[k] : &hd->Wf[k]; ta = &tm_ap; tw = &hd->tm[fp ? 0 : 1].W1[k]; tout = &tm_v;
    } else {
      p.c0 = hd->bg[k]; p.c1 = hd->b2[k]; p.c2 = hd->bsc[k + 1]; p.stats_out = ws.stats; p.h = ws.h; p.out = ws.ap;
      tp = fp ? &hd->Wgs_half[k] : &hd->Wgs[k]; ta = &tm_v; tw = &hd->tm[fp ? 0 : 1].W2[k]; tout = &tm_ap;
    }
    // algorithmic FLOPs: the block's five W x W products are split 2 (first layer and the modulation folded into
    // it; the kernel executes three products) + 3 (gate, next scale, second layer)
    ProfScope ps(ctx, st, kind == FOLD_W1 ? 1 : 3, 2.0 * Rh * static_cast<double>(W) * W * (kind == FOLD_W1 ? 2.0 : 3.0));
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(tiles_n * row_tiles); lc.blockDim = dim3(kFoldThreads); lc.stream = st;
    lc.dynamicSmemBytes = kind == FOLD_W1 ? FoldCfg<FOLD_W1>::kSmemBytes : FoldCfg<FOLD_GATE>::kSmemBytes;
    cudaLaunchAttribute at[2];
    int na = 0;
    if (fp) { at[na].id = cudaLaunchAttributeClusterDimension; at[na].val.clusterDim.x = 2; at[na].val.clusterDim.y = 1; at[na].val.clusterDim.z = 1; ++na; }
    if (!ctx->prof_on) { at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization; at[na].val.programmaticStreamSerializationAllowed = 1; ++na; }
    lc.attrs = at; lc.numAttrs = na;
    const CUtensorMap& ts = tm_sb[cur_t & 1];
#define CSD_FOLD_LAUNCH(ACT, FMT, KIND, PAIR) CSD_CUDA(ctx, cudaLaunchKernelEx(&lc, fold_kernel<ACT, FMT, KIND, PAIR>, ts, *tp, *ta, *tw, *tout, tm_h, tiles_n, p))
    if (d.dtype == CSD_F16) {
      if (kind == FOLD_W1) { if (fp) CSD_FOLD_LAUNCH(__half, 0, FOLD_W1, true); else CSD_FOLD_LAUNCH(__half, 0, FOLD_W1, false); }
      else { if (fp) CSD_FOLD_LAUNCH(__half, 0, FOLD_GATE, true); else CSD_FOLD_LAUNCH(__half, 0, FOLD_GATE, false); }
    } else {
      if (kind == FOLD_W1) { if (fp) CSD_FOLD_LAUNCH(__nv_bfloat16, 1, FOLD_W1, true); else CSD_FOLD_LAUNCH(__nv_bfloat16, 1, FOLD_W1, false); }
      else { if (fp) CSD_FOLD_LAUNCH(__nv_bfloat16, 1, FOLD_GATE, true); else CSD_FOLD_LAUNCH(__nv_bfloat16, 1, FOLD_GATE, false); }
    }
#undef CSD_FOLD_LAUNCH
    ctx->launches++;
    return CSD_OK;
  }

  // The persistent chain kernel: s of every step in the kernel's row order, zeroed counters, the schedule on the
  // device, one launch of CTA pairs.
  int launch_pchain() {
    const csd_head_desc& d = hd->d;
    ChainWs& ws = ctx->ws[slot];
    const size_t asz = 2;
    const int nb0 = cfg ? (R + 63) / 64 : (R + 127) / 128, nb = nb0 + (nb0 & 1);   // row blocks, paired
    const size_t rows = static_cast<size_t>(nb) * kTileM, G = W / kStatCols;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
    const size_t o_s = take(static_cast<size_t>(Ts) * rows * W * asz), o_ap = take(rows * W * asz), o_v = take(rows * W * asz),
                 o_st = take(rows * G * 8), o_ep = take(rows * G * kCPad * 4), o_sync = take(static_cast<size_t>(nb / 2) * 4),
                 o_sched = take(static_cast<size_t>(3) * Ts * 4);
    int rc = ensure_side(ctx, ctx->pc[slot], off, "the persistent chain buffers");
    if (rc) return rc;
    char* b = static_cast<char*>(ctx->pc[slot].base);
    CUtensorMap tm_s{}, tm_a{}, tm_vv{};
    if ((rc = make_tmap(ctx, &tm_s, d.dtype, b + o_s, static_cast<uint64_t>(Ts) * rows, W, W, kTileM))) return rc;
    if ((rc = make_tmap(ctx, &tm_a, d.dtype, b + o_ap, rows, W, W, kTileM))) return rc;
    if ((rc = make_tmap(ctx, &tm_vv, d.dtype, b + o_v, rows, W, W, kTileM))) return rc;
    CSD_CUDA(ctx, cudaMemsetAsync(b + o_sync, 0, static_cast<size_t>(nb / 2) * 4, st));
    float* d_sched = reinterpret_cast<float*>(b + o_sched);
    CSD_CUDA(ctx, cudaMemcpyAsync(d_sched, sc->a, Ts * sizeof(float), cudaMemcpyHostToDevice, st));
    CSD_CUDA(ctx, cudaMemcpyAsync(d_sched + Ts, sc->b, Ts * sizeof(float), cudaMemcpyHostToDevice, st));
    CSD_CUDA(ctx, cudaMemcpyAsync(d_sched + 2 * Ts, sc->sigma, Ts * sizeof(float), cudaMemcpyHostToDevice, st));
    const dim3 sgrid(static_cast<unsigned>(rows), static_cast<unsigned>(Ts));
    if (d.dtype == CSD_F16) pc_cond_all_kernel<__half><<<sgrid, 128, 0, st>>>(ws.cz, ws.te, reinterpret_cast<__half*>(b + o_s), R, cfg, W, static_cast<int>(rows));
    else pc_cond_all_kernel<__nv_bfloat16><<<sgrid, 128, 0, st>>>(ws.cz, ws.te, reinterpret_cast<__nv_bfloat16*>(b + o_s), R, cfg, W, static_cast<int>(rows));
    ctx->launches++;
    CSD_CUDA(ctx, cudaGetLastError());
    PcParams p{};
    p.R = R; p.cfg = cfg; p.W = W; p.L = L; p.T = Ts; p.C = d.C; p.sample_last = sample_last; p.nblk = nb; p.cfg_scale = cfg_scale;
    p.maps = hd->d_pc_maps; p.bias = hd->d_pc_bias; p.sched = d_sched;
    p.win = hd->win; p.bin = hd->bin; p.wout_t = hd->wout_t; p.bout = hd->bout; p.x_T = x_T; p.eps = eps;
    p.x0 = x0; p.mu1 = mu1; p.x1 = x1; p.x = ws.x; p.traj_x = traj_x; p.traj_mu = traj_mu;
    p.stats = reinterpret_cast<float*>(b + o_st); p.epart = reinterpret_cast<float*>(b + o_ep);
    p.sync = reinterpret_cast<unsigned*>(b + o_sync); p.err = ctx->d_err; p.status = ctx->d_err + 1;
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(static_cast<unsigned>(nb) * kPcColTiles); lc.blockDim = dim3(kPcThreads); lc.dynamicSmemBytes = kPcSmemBytes; lc.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    lc.attrs = at; lc.numAttrs = 1;
    if (d.dtype == CSD_F16) CSD_CUDA(ctx, cudaLaunchKernelEx(&lc, pchain_kernel<__half, 0>, tm_s, tm_a, tm_vv, p));
    else CSD_CUDA(ctx, cudaLaunchKernelEx(&lc, pchain_kernel<__nv_bfloat16, 1>, tm_s, tm_a, tm_vv, p));
    ctx->launches++;
    return CSD_OK;
  }

  // The persistent small-batch kernel: s of every step, zeroed counters, the schedule on the device, one launch.
  int launch_small_batch() {
    const csd_head_desc& d = hd->d;
    ChainWs& ws = ctx->ws[slot];
    const size_t asz = 2, nm = static_cast<size_t>(5 * L + 2) * W;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
    const size_t o_s = take(static_cast<size_t>(Ts) * kSbRows * W * asz), o_mods = take(2 * kSbRows * nm * 4),
                 o_ap = take(static_cast<size_t>(kSbRows) * W * asz), o_v = take(static_cast<size_t>(kSbRows) * W * asz),
                 o_sync = take(static_cast<size_t>(Ts + 2) * 4), o_sched = take(static_cast<size_t>(3) * Ts * 4),
                 o_h = take(static_cast<size_t>(kSbRows) * W * 4), o_st = take(static_cast<size_t>(kSbRows) * (W / kStatCols) * 8);
    int rc = ensure_side(ctx, ctx->sb[slot], off, "the small-batch chain buffers");
    if (rc) return rc;
    char* b = static_cast<char*>(ctx->sb[slot].base);
    CUtensorMap tm_a{}, tm_vv{}, tm_sa{};
    if ((rc = make_tmap(ctx, &tm_a, d.dtype, b + o_ap, kSbRows, W, W, kSbGroup))) return rc;     // boxes of one row group
    if ((rc = make_tmap(ctx, &tm_vv, d.dtype, b + o_v, kSbRows, W, W, kSbGroup))) return rc;
    if ((rc = make_tmap(ctx, &tm_sa, d.dtype, b + o_s, static_cast<uint64_t>(Ts) * kSbRows, W, W, kTileM))) return rc;
    CSD_CUDA(ctx, cudaMemsetAsync(b + o_sync, 0, static_cast<size_t>(Ts + 2) * 4, st));
    // small pageable sources: staged by the runtime before the calls return
    float* d_sched = reinterpret_cast<float*>(b + o_sched);
    CSD_CUDA(ctx, cudaMemcpyAsync(d_sched, sc->a, Ts * sizeof(float), cudaMemcpyHostToDevice, st));
    CSD_CUDA(ctx, cudaMemcpyAsync(d_sched + Ts, sc->b, Ts * sizeof(float), cudaMemcpyHostToDevice, st));
    CSD_CUDA(ctx, cudaMemcpyAsync(d_sched + 2 * Ts, sc->sigma, Ts * sizeof(float), cudaMemcpyHostToDevice, st));
    const dim3 sgrid(static_cast<unsigned>(kSbRows), static_cast<unsigned>(Ts));
    if (d.dtype == CSD_F16) sb_cond_all_kernel<__half><<<sgrid, 256, 0, st>>>(ws.cz, ws.te, reinterpret_cast<__half*>(b + o_s), R, cfg, W, Ts);
    else sb_cond_all_kernel<__nv_bfloat16><<<sgrid, 256, 0, st>>>(ws.cz, ws.te, reinterpret_cast<__nv_bfloat16*>(b + o_s), R, cfg, W, Ts);
    ctx->launches++;
    CSD_CUDA(ctx, cudaGetLastError());
    const int ncl = d.dtype == CSD_F16 ? sb_clusters_of<__half, 0>(ctx) : sb_clusters_of<__nv_bfloat16, 1>(ctx);
    SbParams p{};
    p.R = R; p.Rh = Rh; p.cfg = cfg; p.W = W; p.L = L; p.T = Ts; p.C = d.C; p.sample_last = sample_last; p.cfg_scale = cfg_scale;
    const int per = cfg ? 8 : 16;                 // tokens per row group
    p.nd = (R + per - 1) / per; p.ne = ncl - p.nd; p.ntasks = hd->sb_ntasks; p.nm = static_cast<int>(nm);
    p.maps = hd->d_sb_maps; p.tasks = hd->d_sb_tasks; p.sched = d_sched; p.bias = hd->d_sb_bias;
    p.mods = reinterpret_cast<float*>(b + o_mods); p.h = reinterpret_cast<float*>(b + o_h); p.stats = reinterpret_cast<float*>(b + o_st);
    p.ap = b + o_ap; p.v = b + o_v; p.x = ws.x;
    p.win = hd->win; p.bin = hd->bin; p.wout_t = hd->wout_t; p.bout = hd->bout; p.x_T = x_T; p.eps = eps;
    p.x0 = x0; p.mu1 = mu1; p.x1 = x1; p.sync = reinterpret_cast<int*>(b + o_sync); p.err = ctx->d_err; p.status = ctx->d_err + 1;
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3((p.nd + p.ne) * kSbCluster); lc.blockDim = dim3(kSbThreads); lc.dynamicSmemBytes = kSbSmemBytes; lc.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = kSbCluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    lc.attrs = at; lc.numAttrs = 1;
    if (d.dtype == CSD_F16) CSD_CUDA(ctx, cudaLaunchKernelEx(&lc, sb_chain_kernel<__half, 0>, tm_a, tm_vv, tm_sa, p));
    else CSD_CUDA(ctx, cudaLaunchKernelEx(&lc, sb_chain_kernel<__nv_bfloat16, 1>, tm_a, tm_vv, tm_sa, p));
    ctx->launches++;
    return CSD_OK;
  }

  int step(int t) {
    if (sbk || pck) return CSD_OK;   // already enqueued by begin()
    const csd_head_desc& d = hd->d;
    ChainWs& ws = ctx->ws[slot];
    cur_t = t;
    const CUtensorMap& tm_s = tm_sb[t & 1];
    const float* sf = static_cast<const float*>(sbuf[t & 1]);
    const float* uf = static_cast<const float*>(ws.u);
    const float* vf = static_cast<const float*>(ws.v);
    const csd_head::TmSet& tmw = hd->tm[(tn == 64 || pair) ? 0 : 1];   // pairs load half of each B tile per CTA
    int rc = CSD_OK;
    for (int k = 0; k < L; ++k) {
      EpiParams e = ep;
      e.h = ws.h; e.stats = ws.stats;
      const bool folded_in = fold && k >= 1;        // the block's input is a' = h (1 + scale): no modulate kernel
      const bool folded_out = fold && k + 1 < L;    // the block's last kernel also forms a' of the next block
      if (folded_in) {
        if ((rc = launch_fold(FOLD_W1, k))) return rc;
        if (folded_out) rc = launch_fold(FOLD_GATE, k);
        if (rc) return rc;
        if (folded_out) continue;
      }
      // u = LN(h)(1 + scale) + shift
      e.bias0 = hd->bsh[k]; e.bias1 = hd->bsc[k]; e.out_act = ws.u;
      // s of the first step is written by the kernel right before the first modulate kernel; every later s is older
      const int dep_mod = (k == 0 && t == T) ? 0 : W;
      if (folded_in) rc = CSD_OK;
      else if (tc && mod64) rc = launch_tc<EPI_MOD, 1, 2>(ctx, d.dtype, 64, false, st, tm_s, hd->tm[0].Wss[k], tm_s, hd->tm[0].Wss[k], tm_h, W, 0, dep_mod, W, e, &tm_u);
      else if (tc) rc = launch_tc<EPI_MOD, 1, 2>(ctx, d.dtype, tn, pair, st, tm_s, tmw.Wss[k], tm_s, tmw.Wss[k], tm_h, W, 0, dep_mod, W, e, &tm_u);
      else rc = launch_simt<EPI_MOD, 1, 256>(ctx, st, sf, W, static_cast<const float*>(hd->Wss[k]), W, nullptr, 0,
                                             nullptr, 0, W, e);
      if (rc) return rc;
      // v = SiLU(W1 u + b1)
      e.bias0 = hd->b1[k]; e.bias1 = nullptr; e.out_act = ws.v;
      if (folded_in) rc = CSD_OK;
      else if (tc && pair && W % 256 == 0) {
        // CTA pairs over 256 x 256 tiles: per MMA byte the pair loads half as many operand bytes as with 256 x 128
        // tiles, and the first layer (one accumulator, K = W) is the kernel bound by that feed
        const CUtensorMap& w1 = hd->tm[1].W1[k];   // 128-row boxes: each CTA of the pair loads half of the 256 rows
        rc = d.dtype == CSD_F16 ? launch_tc_t<EPI_SILU_ACT, 1, 1, 256, __half, true>(ctx, st, tm_u, w1, tm_u, w1, tm_h, W, 0, 0, W, e, &tm_v)
                                : launch_tc_t<EPI_SILU_ACT, 1, 1, 256, __nv_bfloat16, true>(ctx, st, tm_u, w1, tm_u, w1, tm_h, W, 0, 0, W, e, &tm_v);
      }
      else if (tc && w1_wide) {
        const CUtensorMap& w1 = hd->W1_wide[k];
        rc = d.dtype == CSD_F16 ? launch_tc_t<EPI_SILU_ACT, 1, 1, 256, __half, false>(ctx, st, tm_u, w1, tm_u, w1, tm_h, W, 0, 0, W, e, &tm_v)
                                : launch_tc_t<EPI_SILU_ACT, 1, 1, 256, __nv_bfloat16, false>(ctx, st, tm_u, w1, tm_u, w1, tm_h, W, 0, 0, W, e, &tm_v);
      }
      else if (tc) rc = launch_tc<EPI_SILU_ACT, 1, 1>(ctx, d.dtype, tn, pair, st, tm_u, tmw.W1[k], tm_u, tmw.W1[k], tm_h, W, 0, 0, W, e, &tm_v);
      else rc = launch_simt<EPI_SILU_ACT, 1, 128>(ctx, st, uf, W, static_cast<const float*>(hd->W1[k]), W, nullptr, 0,
                                                  nullptr, 0, W, e);
      if (rc) return rc;
      // h += gate * (W2 v + b2).  On the tensor-core path the gate product s Wg^T comes first: it does
      // not depend on the preceding kernel (which writes v) and overlaps with it.
      e.bias0 = hd->b2[k]; e.bias1 = hd->bg[k]; e.out_act = nullptr;
      if (folded_out) rc = launch_fold(FOLD_GATE, k);
      else if (tc) {
        EpiParams g = e;
        g.bias0 = hd->bg[k]; g.bias1 = hd->b2[k];
        rc = launch_tc<EPI_GATE_RES, 2, 1>(ctx, d.dtype, tn, pair, st, tm_s, tmw.Wg[k], tm_v, tmw.W2[k], tm_h, W, W, W, W, g);
      }
      else rc = launch_simt<EPI_GATE_RES, 2, 128>(ctx, st, vf, W, static_cast<const float*>(hd->W2[k]), W, sf, W,
                                                  static_cast<const float*>(hd->Wg[k]), W, W, e);
      if (rc) return rc;
    }
    EpiParams e = ep;
    e.h = ws.h; e.stats = ws.stats; e.bias0 = hd->bfsh; e.bias1 = hd->bfsc; e.wout_t = hd->wout_t; e.epart = ws.epart;
    if (d.var_out) {   // 32 output columns: eps_hat | variance parameter
      if (tc && mod64) rc = launch_tc<EPI_MODF2, 1, 2>(ctx, d.dtype, 64, false, st, tm_s, hd->tm[0].Wfss, tm_s, hd->tm[0].Wfss, tm_h, W, 0, W, W, e);
      else if (tc) rc = launch_tc<EPI_MODF2, 1, 2>(ctx, d.dtype, tn, pair, st, tm_s, tmw.Wfss, tm_s, tmw.Wfss, tm_h, W, 0, W, W, e);
      else rc = launch_simt<EPI_MODF2, 1, 256>(ctx, st, sf, W, static_cast<const float*>(hd->Wfss), W, nullptr, 0, nullptr,
                                               0, W, e);
    }
    else if (tc && mod64) rc = launch_tc<EPI_MODF, 1, 2>(ctx, d.dtype, 64, false, st, tm_s, hd->tm[0].Wfss, tm_s, hd->tm[0].Wfss, tm_h, W, 0, W, W, e);
    else if (tc) rc = launch_tc<EPI_MODF, 1, 2>(ctx, d.dtype, tn, pair, st, tm_s, tmw.Wfss, tm_s, tmw.Wfss, tm_h, W, 0, W, W, e);
    else rc = launch_simt<EPI_MODF, 1, 256>(ctx, st, sf, W, static_cast<const float*>(hd->Wfss), W, nullptr, 0, nullptr,
                                            0, W, e);
    if (rc) return rc;
    if (batch_Rin) return launch_batch(1);
    if (traj_x) {   // slot j holds x_{T-j} and mu_{T-j}: this boundary produces x_{t-1} and mu_t
      sp.traj_x = traj_x + static_cast<size_t>(T - t + 1) * R * d.C;
      sp.traj_mu = traj_mu + static_cast<size_t>(T - t) * R * d.C;
    }
    sp.a = sc->a[t - 1]; sp.b = sc->b[t - 1];
    if (lv_min) { sp.sigma = 0.0f; sp.lv_min = lv_min[t - 1]; sp.lv_max = lv_max[t - 1]; }
    else sp.sigma = sc->sigma[t - 1];
    sp.eps_t = eps + static_cast<size_t>(t - 1) * R * d.C;
    // this boundary prepares h of step t - 1 and s of step t - 2
    sp.s = t >= 3 ? sbuf[(t - 2) & 1] : nullptr;
    if (t >= 3) sp.te_next = ws.te + static_cast<size_t>(t - 3) * W;
    sp.s_b = nullptr; sp.te_b = nullptr;
    return launch_step(t > 1 ? STEP_MID : STEP_LAST);
  }
};

int run_chain(csd_ctx* ctx, int slot, cudaStream_t st, const csd_head* hd, const csd_schedule* sc, int R, int cfg,
              float cfg_scale, const float* z, const float* x_T, const float* eps, int sample_last, float* x0,
              float* mu1, float* x1) {
  Chain c{ctx, slot, st, hd, sc, R, cfg, cfg_scale, z, x_T, eps, sample_last, x0, mu1, x1};
  int rc = c.begin();
  for (int t = sc->T; t >= 1 && !rc; --t) rc = c.step(t);
  return rc;
}

int check_chain_args(csd_ctx* ctx, const csd_head* hd, const csd_schedule* sc, int R, int cfg, const void* z,
                     const void* x_T, const void* eps) {
  if (!hd) return fail(ctx, CSD_ERR_INVALID_ARG, "head is null");
  if (hd->ctx != ctx) return fail(ctx, CSD_ERR_INVALID_ARG, "head belongs to another context");
  if (hd->d.var_out) return fail(ctx, CSD_ERR_UNSUPPORTED, "this head predicts its variances (var_out = 1): use the _lv calls");
  int rc = check_sched(ctx, sc, true);
  if (rc) return rc;
  if (R < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "row count %d must be >= 1", R);
  if (cfg != 0 && cfg != 1) return fail(ctx, CSD_ERR_INVALID_ARG, "cfg must be 0 or 1");
  if (!z || !x_T || !eps) return fail(ctx, CSD_ERR_INVALID_ARG, "z / x_T / eps is null");
  return CSD_OK;
}

int check_lv_args(csd_ctx* ctx, const csd_head* hd, const csd_schedule_lv* sc, int R, int cfg, const void* z,
                  const void* x_T, const void* eps) {
  if (!hd) return fail(ctx, CSD_ERR_INVALID_ARG, "head is null");
  if (hd->ctx != ctx) return fail(ctx, CSD_ERR_INVALID_ARG, "head belongs to another context");
  if (!hd->d.var_out) return fail(ctx, CSD_ERR_UNSUPPORTED, "this head has a fixed variance (var_out = 0): use the calls without _lv");
  if (!sc) return fail(ctx, CSD_ERR_INVALID_ARG, "schedule is null");
  if (sc->T < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "schedule T = %d must be >= 1", sc->T);
  if (!sc->a || !sc->b || !sc->lv_min || !sc->lv_max || !sc->tfeat) return fail(ctx, CSD_ERR_INVALID_ARG, "schedule a / b / lv_min / lv_max / tfeat is null");
  for (int t = 0; t < sc->T; ++t)
    if (!(sc->lv_min[t] <= sc->lv_max[t]) || !std::isfinite(sc->lv_min[t]) || !std::isfinite(sc->lv_max[t]))
      return fail(ctx, CSD_ERR_INVALID_ARG, "schedule needs finite lv_min[%d] <= lv_max[%d]", t, t);
  if (R < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "row count %d must be >= 1", R);
  if (cfg != 0 && cfg != 1) return fail(ctx, CSD_ERR_INVALID_ARG, "cfg must be 0 or 1");
  if (!z || !x_T || !eps) return fail(ctx, CSD_ERR_INVALID_ARG, "z / x_T / eps is null");
  return CSD_OK;
}

// A learned-variance chain: the fixed-variance chain with the log-variance bounds in place of sigma.
Chain make_lv_chain(csd_ctx* ctx, int slot, cudaStream_t st, const csd_head* hd, const csd_schedule* view,
                    const csd_schedule_lv* sc, int R, int cfg, float cfg_scale, const float* z, const float* x_T,
                    const float* eps, int sample_last, float* x0, float* mu1, float* lv1, float* half_logdet, float* x1) {
  Chain c{ctx, slot, st, hd, view, R, cfg, cfg_scale, z, x_T, eps, sample_last, x0, mu1, x1};
  c.lv_min = sc->lv_min; c.lv_max = sc->lv_max; c.lv1 = lv1; c.half_logdet = half_logdet;
  return c;
}

int accept_scan_lv(csd_ctx* ctx, cudaStream_t st, int B, int gamma, int C, const float* x0, const float* mu_q,
                   const float* lv_q, const float* hld_q, const float* mu_p, const float* lv_p, const float* hld_p,
                   const float* u, float* logratio, float* log_sigma_rows, int32_t* n_accept, uint32_t* mask) {
  accept_scan_lv_kernel<<<(B + 3) / 4, 128, 0, st>>>(B, gamma, C, x0, mu_q, lv_q, hld_q, mu_p, lv_p, hld_p, u, logratio,
                                                     log_sigma_rows, n_accept, mask);
  ctx->launches++;
  CSD_CUDA(ctx, cudaGetLastError());
  return CSD_OK;
}

int resample_lv(csd_ctx* ctx, cudaStream_t st, int B, int gamma, int C, int cap, const float* log_sigma_rows,
                const int32_t* n_accept, const float* mu_p, const float* lv_p, const float* mu_q, const float* lv_q,
                const float* xi, const float* v, float* x_new, int32_t* n_prop, uint32_t* flags, int32_t* cap_hits) {
  CSD_CUDA(ctx, cudaMemsetAsync(cap_hits, 0, sizeof(int32_t), st));
  resample_lv_kernel<<<(B + 3) / 4, 128, 0, st>>>(B, gamma, C, cap, log_sigma_rows, n_accept, mu_p, lv_p, mu_q, lv_q, xi, v,
                                                  x_new, n_prop, flags, cap_hits);
  ctx->launches++;
  CSD_CUDA(ctx, cudaGetLastError());
  return CSD_OK;
}

double log_sigma_term(const csd_schedule* q, const csd_schedule* p, int C) {
  double acc = 0.0;
  for (int t = 1; t < q->T; ++t) acc += std::log(static_cast<double>(q->sigma[t])) - std::log(static_cast<double>(p->sigma[t]));
  return C * acc;
}

int accept_scan(csd_ctx* ctx, cudaStream_t st, int B, int gamma, int C, double log_sigma, float sp1, float sq1,
                const float* x0, const float* mu_q, const float* mu_p, const float* u, float* logratio,
                int32_t* n_accept, uint32_t* mask, const float* offset = nullptr) {
  const double lc = log_sigma + C * (std::log(static_cast<double>(sq1)) - std::log(static_cast<double>(sp1)));
  const float inv2vp = static_cast<float>(0.5 / (static_cast<double>(sp1) * sp1));
  const float inv2vq = static_cast<float>(0.5 / (static_cast<double>(sq1) * sq1));
  accept_scan_kernel<<<(B + 3) / 4, 128, 0, st>>>(B, gamma, C, static_cast<float>(lc), inv2vp, inv2vq, x0, mu_q, mu_p, u,
                                                  logratio, n_accept, mask, offset);
  ctx->launches++;
  CSD_CUDA(ctx, cudaGetLastError());
  return CSD_OK;
}

int resample(csd_ctx* ctx, cudaStream_t st, int B, int gamma, int C, int cap, double log_sigma, float sp1, float sq1,
             const int32_t* n_accept, const float* mu_p, const float* mu_q, const float* xi, const float* v,
             float* x_new, int32_t* n_prop, uint32_t* flags, int32_t* cap_hits) {
  CSD_CUDA(ctx, cudaMemsetAsync(cap_hits, 0, sizeof(int32_t), st));
  resample_kernel<<<(B + 3) / 4, 128, 0, st>>>(B, gamma, C, cap, static_cast<float>(log_sigma), sp1, sq1,
                                               static_cast<float>(std::log(static_cast<double>(sp1))),
                                               static_cast<float>(std::log(static_cast<double>(sq1))), n_accept, mu_p,
                                               mu_q, xi, v, x_new, n_prop, flags, cap_hits);
  ctx->launches++;
  CSD_CUDA(ctx, cudaGetLastError());
  return CSD_OK;
}

// Target chain over the R = B gamma verified positions with the B rows of position gamma + 1 appended (Alg. 1
// obtains p_{gamma+1} from the same parallel target pass): token rows [0, R) are the verified ones, [R, R + B) the
// bonus ones; with guidance the unconditional twins follow in the same order.  The side buffer holds the gathered
// inputs and the chain's last-step outputs for all R + B rows.
struct BonusBuf {
  float *z, *x_T, *eps, *mu1, *x0;
};

size_t bonus_buf_bytes(const csd_head_desc& d, int Rt, int cfg, int T) {
  const size_t m = cfg ? 2 : 1, rt = static_cast<size_t>(Rt);
  return align_up(rt * m * d.Dz * 4, 256) + align_up(rt * d.C * 4, 256) * 3 + align_up(static_cast<size_t>(T) * rt * d.C * 4, 256);
}

int ensure_side(csd_ctx* ctx, HostIo& io, size_t need, const char* what) {
  if (need <= io.cap) return CSD_OK;
  CSD_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  for (int i = 0; i < 2; ++i) CSD_CUDA(ctx, cudaStreamSynchronize(ctx->side[i]));
  if (io.base) CSD_CUDA(ctx, cudaFree(io.base));
  io.base = nullptr; io.cap = 0;
  if (cudaMalloc(&io.base, need) != cudaSuccess) {
    cudaGetLastError();
    return fail(ctx, CSD_ERR_WORKSPACE, "cannot allocate %zu bytes for %s", need, what);
  }
  io.cap = need;
  return CSD_OK;
}

// Carves the (already large enough) side buffer and enqueues the gathering copies on `st`.
int gather_bonus_inputs(csd_ctx* ctx, cudaStream_t st, const csd_head_desc& d, int R, int B, int cfg, int T,
                        const float* z, const float* x_T, const float* eps, const float* z_next,
                        const float* x_T_next, const float* eps_next, BonusBuf& bb) {
  const size_t m = cfg ? 2 : 1, Rt = static_cast<size_t>(R) + B, C = d.C, Dz = d.Dz;
  char* p = static_cast<char*>(ctx->bn.base);
  bb.z = reinterpret_cast<float*>(p); p += align_up(Rt * m * Dz * 4, 256);
  bb.x_T = reinterpret_cast<float*>(p); p += align_up(Rt * C * 4, 256);
  bb.mu1 = reinterpret_cast<float*>(p); p += align_up(Rt * C * 4, 256);
  bb.x0 = reinterpret_cast<float*>(p); p += align_up(Rt * C * 4, 256);
  bb.eps = reinterpret_cast<float*>(p);
  for (size_t h = 0; h < m; ++h) {
    CSD_CUDA(ctx, cudaMemcpyAsync(bb.z + h * Rt * Dz, z + h * R * Dz, static_cast<size_t>(R) * Dz * 4, cudaMemcpyDeviceToDevice, st));
    CSD_CUDA(ctx, cudaMemcpyAsync(bb.z + (h * Rt + R) * Dz, z_next + h * B * Dz, static_cast<size_t>(B) * Dz * 4, cudaMemcpyDeviceToDevice, st));
  }
  CSD_CUDA(ctx, cudaMemcpyAsync(bb.x_T, x_T, static_cast<size_t>(R) * C * 4, cudaMemcpyDeviceToDevice, st));
  CSD_CUDA(ctx, cudaMemcpyAsync(bb.x_T + static_cast<size_t>(R) * C, x_T_next, static_cast<size_t>(B) * C * 4, cudaMemcpyDeviceToDevice, st));
  CSD_CUDA(ctx, cudaMemcpy2DAsync(bb.eps, Rt * C * 4, eps, static_cast<size_t>(R) * C * 4, static_cast<size_t>(R) * C * 4, T, cudaMemcpyDeviceToDevice, st));
  CSD_CUDA(ctx, cudaMemcpy2DAsync(bb.eps + static_cast<size_t>(R) * C, Rt * C * 4, eps_next, static_cast<size_t>(B) * C * 4, static_cast<size_t>(B) * C * 4, T, cudaMemcpyDeviceToDevice, st));
  return CSD_OK;
}

int check_verify_dims(csd_ctx* ctx, int B, int gamma, int C) {
  if (B < 1 || gamma < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "B = %d and gamma = %d must be >= 1", B, gamma);
  if (gamma > 32) return fail(ctx, CSD_ERR_UNSUPPORTED, "gamma = %d exceeds 32", gamma);
  if (C < 1 || C > kCPad) return fail(ctx, CSD_ERR_UNSUPPORTED, "token dim C = %d must be in [1, 16]", C);
  return CSD_OK;
}

}  // namespace

// ================================================================================== C ABI
extern "C" {

int csd_create(csd_ctx** out, int device, void* cuda_stream) {
  if (!out) return CSD_ERR_INVALID_ARG;
  *out = nullptr;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
    cudaGetLastError();
    return CSD_ERR_CUDA;
  }
  if (device >= kMaxDevices) return CSD_ERR_UNSUPPORTED;
  DeviceGuard dg(device);   // the caller's current device is put back when this call returns
  if (!dg.ok) return CSD_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return CSD_ERR_CUDA;
  if (prop.major != 10) return CSD_ERR_UNSUPPORTED;  // kernels are built for sm_100a only
  csd_ctx* c = new (std::nothrow) csd_ctx();
  if (!c) return CSD_ERR_WORKSPACE;
  c->device = device;
  c->num_sms = prop.multiProcessorCount;
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  bool ok = true;
  // side[1] outranks side[0]: csd_round puts the longer of its two chains there, so that the chain that decides
  // the round's duration gets free SMs first and the shorter one fills the gaps
  int prio_lo = 0, prio_hi = 0;
  cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);
  for (int i = 0; i < 2; ++i) {
    ok = ok && cudaStreamCreateWithPriority(&c->side[i], cudaStreamNonBlocking, i == 1 ? prio_hi : prio_lo) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->ev_done[i], cudaEventDisableTiming) == cudaSuccess;
  }
  ok = ok && cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_err, 2 * sizeof(int)) == cudaSuccess;   // [0] first failed wait, [1] non-finite value seen
  ok = ok && cudaMemset(c->d_err, 0, 2 * sizeof(int)) == cudaSuccess;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  ok = ok && cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
       qres == cudaDriverEntryPointSuccess && fn != nullptr;
  if (!ok) {
    cudaGetLastError();
    csd_destroy(c);
    return CSD_ERR_CUDA;
  }
  c->encode = reinterpret_cast<EncodeTiledFn>(fn);
  *out = c;
  return CSD_OK;
}

int csd_destroy(csd_ctx* c) {
  if (!c) return CSD_ERR_INVALID_ARG;
  DeviceGuard dg(c->device);
  cudaStreamSynchronize(c->stream);
  for (int i = 0; i < 2; ++i) {
    if (c->side[i]) { cudaStreamSynchronize(c->side[i]); cudaStreamDestroy(c->side[i]); }
    if (c->ev_done[i]) cudaEventDestroy(c->ev_done[i]);
  }
  for (ChainWs& w : c->ws)
    if (w.base && w.owned) cudaFree(w.base);
  for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->io.base) cudaFree(c->io.base);
  if (c->sp.base) cudaFree(c->sp.base);
  if (c->un.base) cudaFree(c->un.base);
  if (c->bn.base) cudaFree(c->bn.base);
  for (HostIo& b : c->sb) if (b.base) cudaFree(b.base);
  for (HostIo& b : c->pc) if (b.base) cudaFree(b.base);
  if (c->d_err) cudaFree(c->d_err);
  cudaGetLastError();
  delete c;
  return CSD_OK;
}

const char* csd_last_error(const csd_ctx* c) { return c ? c->err : "null context"; }

int64_t csd_launch_count(const csd_ctx* c) { return c ? c->launches : 0; }

int csd_sync(csd_ctx* c) {
  if (!c) return CSD_ERR_INVALID_ARG;
  CSD_DEVICE(c);
  CSD_CUDA(c, cudaStreamSynchronize(c->stream));
  int e[2] = {0, 0};
  CSD_CUDA(c, cudaMemcpy(e, c->d_err, sizeof(e), cudaMemcpyDeviceToHost));
  if (e[0] != 0 || e[1] != 0) cudaMemset(c->d_err, 0, sizeof(e));
  if (e[0] != 0) {
    static const char* const roles[] = {"?", "TMA producer", "MMA issuer", "epilogue", "wait self-test"};
    const int role = e[0] & 0xf;
    return fail(c, CSD_ERR_TIMEOUT, "a device-side bounded wait gave up: %s (role %d), site %d, iteration %d, block %d",
                roles[role <= 4 ? role : 0], role, (e[0] >> 4) & 0xf, (e[0] >> 8) & 0xffff, (e[0] >> 24) & 0x7f);
  }
  if (e[1] != 0)
    return fail(c, CSD_ERR_NONFINITE, "a non-finite value reached a step update: an activation beyond the operand "
                "format's range (65504 for CSD_F16 heads: use CSD_BF16 or CSD_F32) or non-finite inputs");
  return CSD_OK;
}

int csd_set_wait_limit(csd_ctx* c, int64_t cycles) {
  if (!c) return CSD_ERR_INVALID_ARG;
  CSD_DEVICE(c);
  CSD_CUDA(c, cudaStreamSynchronize(c->stream));
  for (int i = 0; i < 2; ++i) CSD_CUDA(c, cudaStreamSynchronize(c->side[i]));
  const long long v = cycles > 0 ? static_cast<long long>(cycles) : 4000000000ll;
  CSD_CUDA(c, cudaMemcpyToSymbol(g_wait_limit_cycles, &v, sizeof(v)));
  return CSD_OK;
}

int csd_selftest_wait_timeout(csd_ctx* c) {
  if (!c) return CSD_ERR_INVALID_ARG;
  CSD_DEVICE(c);
  wait_timeout_selftest_kernel<<<1, 32, 0, c->stream>>>(c->d_err);
  c->launches++;
  CSD_CUDA(c, cudaGetLastError());
  return CSD_OK;
}

int csd_set_chain_mode(csd_ctx* c, int mode) {
  if (!c) return CSD_ERR_INVALID_ARG;
  if (mode != CSD_CHAIN_LAYERS && mode != CSD_CHAIN_LAYERS_PLAIN && mode != CSD_CHAIN_SMALL_BATCH && mode != CSD_CHAIN_LAYER_KERNELS) return fail(c, CSD_ERR_INVALID_ARG, "chain mode %d unknown", mode);
  c->chain_mode = mode;
  return CSD_OK;
}

int csd_profile(csd_ctx* c, int enable) {
  if (!c) return CSD_ERR_INVALID_ARG;
  CSD_DEVICE(c);
  CSD_CUDA(c, cudaStreamSynchronize(c->stream));
  c->prof_on = enable != 0;
  c->prof.clear();
  c->ev_used = 0;
  return CSD_OK;
}

int csd_profile_read(csd_ctx* c, int kernel_class, int64_t* launches, double* total_ms, double* total_flops) {
  if (!c) return CSD_ERR_INVALID_ARG;
  if (!launches || !total_ms || !total_flops) return fail(c, CSD_ERR_INVALID_ARG, "null output pointer");
  if (kernel_class < 0 || kernel_class > 6) return fail(c, CSD_ERR_INVALID_ARG, "kernel class %d not in [0, 6]", kernel_class);
  CSD_DEVICE(c);
  CSD_CUDA(c, cudaStreamSynchronize(c->stream));
  for (int i = 0; i < 2; ++i) CSD_CUDA(c, cudaStreamSynchronize(c->side[i]));
  *launches = 0; *total_ms = 0.0; *total_flops = 0.0;
  for (const ProfRec& r : c->prof) {
    if (r.cls != kernel_class) continue;
    float ms = 0.0f;
    CSD_CUDA(c, cudaEventElapsedTime(&ms, r.a, r.b));
    *launches += 1; *total_ms += ms; *total_flops += r.flops;
  }
  return CSD_OK;
}

int csd_schedule_ddpm(int T, const double* beta, double tau, float* a, float* b, float* sigma) {
  if (T < 1 || !beta || !a || !b || !sigma || !(tau > 0.0)) return CSD_ERR_INVALID_ARG;
  double abar = 1.0;
  for (int t = 0; t < T; ++t) {
    if (!(beta[t] > 0.0 && beta[t] < 1.0)) return CSD_ERR_INVALID_ARG;
    const double alpha = 1.0 - beta[t];
    abar *= alpha;
    a[t] = static_cast<float>(1.0 / std::sqrt(alpha));
    b[t] = static_cast<float>(beta[t] / (std::sqrt(alpha) * std::sqrt(1.0 - abar)));
    sigma[t] = static_cast<float>(tau * std::sqrt(beta[t]));
  }
  return CSD_OK;
}

int csd_schedule_ddim(int T_full, const double* beta_full, int n_steps, const int32_t* steps, double eta, float* a,
                      float* b, float* sigma) {
  if (T_full < 1 || n_steps < 1 || !beta_full || !steps || !a || !b || !sigma) return CSD_ERR_INVALID_ARG;
  if (!(eta > 0.0 && eta <= 1.0)) return CSD_ERR_INVALID_ARG;
  std::vector<double> abar(static_cast<size_t>(T_full));
  double acc = 1.0;
  for (int t = 0; t < T_full; ++t) {
    if (!(beta_full[t] > 0.0 && beta_full[t] < 1.0)) return CSD_ERR_INVALID_ARG;
    acc *= 1.0 - beta_full[t];
    abar[t] = acc;
  }
  for (int k = 0; k < n_steps; ++k) {
    if (steps[k] < 1 || steps[k] > T_full || (k > 0 && steps[k] <= steps[k - 1])) return CSD_ERR_INVALID_ARG;
    const double cur = abar[steps[k] - 1], prv = k > 0 ? abar[steps[k - 1] - 1] : 1.0;
    // variance of q_sigma(x_prev | x_t, x0_hat); the step to x_0 would have none (prv = 1): it gets the
    // variance of the chain's own forward step around the predicted x_0
    const double sg = k > 0 ? eta * std::sqrt((1.0 - prv) / (1.0 - cur)) * std::sqrt(1.0 - cur / prv) : eta * std::sqrt(1.0 - cur);
    const double keep = k > 0 ? std::sqrt(std::fmax(0.0, 1.0 - prv - sg * sg)) : 0.0;   // weight of eps_hat towards x_t
    const double scale = std::sqrt(prv / cur);
    a[k] = static_cast<float>(scale);
    b[k] = static_cast<float>(scale * std::sqrt(1.0 - cur) - keep);
    sigma[k] = static_cast<float>(sg);
  }
  return CSD_OK;
}

int csd_log_sigma_term(int T, const float* sigma_q, const float* sigma_p, int C, double* out) {
  if (T < 1 || C < 1 || !sigma_q || !sigma_p || !out) return CSD_ERR_INVALID_ARG;
  for (int t = 0; t < T; ++t)
    if (!(sigma_q[t] > 0.0f) || !(sigma_p[t] > 0.0f)) return CSD_ERR_INVALID_ARG;
  csd_schedule q{}, p{};
  q.T = T; q.sigma = sigma_q; p.T = T; p.sigma = sigma_p;
  *out = log_sigma_term(&q, &p, C);
  return CSD_OK;
}

int csd_head_create(csd_ctx* ctx, const csd_head_desc* desc, const csd_head_weights* w, csd_head** out) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  if (!desc || !w || !out) return fail(ctx, CSD_ERR_INVALID_ARG, "desc / weights / out is null");
  *out = nullptr;
  const csd_head_desc d = *desc;
  if (d.dtype != CSD_F32 && d.dtype != CSD_BF16 && d.dtype != CSD_F16) return fail(ctx, CSD_ERR_INVALID_ARG, "dtype %d unknown", d.dtype);
  if (d.C < 1 || d.W < 1 || d.L < 1 || d.Dz < 1 || d.F < 1)
    return fail(ctx, CSD_ERR_INVALID_ARG, "head dims must be positive (C=%d W=%d L=%d Dz=%d F=%d)", d.C, d.W, d.L, d.Dz, d.F);
  if (d.C > kCPad) return fail(ctx, CSD_ERR_UNSUPPORTED, "token dim C = %d exceeds 16", d.C);
  if (d.var_out != 0 && d.var_out != 1) return fail(ctx, CSD_ERR_INVALID_ARG, "var_out = %d must be 0 or 1", d.var_out);
  if (d.W % kTileN != 0) return fail(ctx, CSD_ERR_UNSUPPORTED, "width W = %d must be a multiple of 128", d.W);
  const int kmul = d.dtype != CSD_F32 ? kBlockK : kSimtBK;
  if (d.Dz % kmul != 0) return fail(ctx, CSD_ERR_UNSUPPORTED, "Dz = %d must be a multiple of %d", d.Dz, kmul);
  const float* const* ptrs = reinterpret_cast<const float* const*>(w);
  for (size_t i = 0; i < sizeof(csd_head_weights) / sizeof(float*); ++i)
    if (!ptrs[i]) return fail(ctx, CSD_ERR_INVALID_ARG, "weight pointer #%zu is null", i);
  CSD_DEVICE(ctx);

  csd_head* h = new (std::nothrow) csd_head();
  if (!h) return fail(ctx, CSD_ERR_WORKSPACE, "out of host memory");
  h->ctx = ctx; h->d = d; h->esz = d.dtype != CSD_F32 ? 2 : 4;
  const size_t W = d.W, L = d.L, Dz = d.Dz, F = d.F, C = d.C;

  // ---- GEMM weights, packed: Wz | per block (Wss, Wg, W1, W2) | Wfss
  const size_t n_gemm = W * Dz + L * (5 * W * W) + 2 * W * W;
  std::vector<float> stage;
  try { stage.resize(n_gemm); } catch (...) { delete h; return fail(ctx, CSD_ERR_WORKSPACE, "out of host memory"); }
  std::vector<size_t> o_wss(L), o_wg(L), o_w1(L), o_w2(L);
  size_t off = 0;
  const size_t o_wz = off; memcpy(&stage[off], w->Wz, W * Dz * 4); off += W * Dz;
  // AdaLN shift and scale rows interleaved in groups of 64: 64 shift rows | 64 scale rows | ...
  auto interleave = [&](const float* shift_rows, const float* scale_rows, float* dst) {
    for (size_t j = 0; j < W / kStatCols; ++j) {
      memcpy(dst + (2 * j) * kStatCols * W, shift_rows + j * kStatCols * W, kStatCols * W * 4);
      memcpy(dst + (2 * j + 1) * kStatCols * W, scale_rows + j * kStatCols * W, kStatCols * W * 4);
    }
  };
  for (size_t k = 0; k < L; ++k) {
    const float* ada = w->Wada + k * 3 * W * W;
    o_wss[k] = off; interleave(ada, ada + W * W, &stage[off]); off += 2 * W * W;
    o_wg[k] = off; memcpy(&stage[off], ada + 2 * W * W, W * W * 4); off += W * W;
    o_w1[k] = off; memcpy(&stage[off], w->W1 + k * W * W, W * W * 4); off += W * W;
    o_w2[k] = off; memcpy(&stage[off], w->W2 + k * W * W, W * W * 4); off += W * W;
  }
  const size_t o_wfss = off; interleave(w->Wfada, w->Wfada + W * W, &stage[off]); off += 2 * W * W;

  auto bail = [&](int code, const char* what) { csd_head_destroy(h); return fail(ctx, code, "%s", what); };
  if (cudaMalloc(&h->wblob, n_gemm * h->esz) != cudaSuccess) { cudaGetLastError(); return bail(CSD_ERR_WORKSPACE, "cannot allocate device memory for the weights"); }
  if (d.dtype != CSD_F32) {
    std::vector<uint16_t> hb;
    try { hb.resize(n_gemm); } catch (...) { return bail(CSD_ERR_WORKSPACE, "out of host memory"); }
    if (d.dtype == CSD_BF16) {
      for (size_t i = 0; i < n_gemm; ++i) hb[i] = f32_to_bf16_bits(stage[i]);
    } else {
      for (size_t i = 0; i < n_gemm; ++i) { const __half hv = __float2half_rn(stage[i]); memcpy(&hb[i], &hv, 2); }
    }
    if (cudaMemcpy(h->wblob, hb.data(), n_gemm * 2, cudaMemcpyHostToDevice) != cudaSuccess) return bail(CSD_ERR_CUDA, "weight upload failed");
  } else {
    if (cudaMemcpy(h->wblob, stage.data(), n_gemm * 4, cudaMemcpyHostToDevice) != cudaSuccess) return bail(CSD_ERR_CUDA, "weight upload failed");
  }
  auto wp = [&](size_t o) { return static_cast<void*>(static_cast<char*>(h->wblob) + o * h->esz); };
  h->Wz = wp(o_wz); h->Wfss = wp(o_wfss);
  h->Wss.resize(L); h->Wg.resize(L); h->W1.resize(L); h->W2.resize(L);
  for (size_t k = 0; k < L; ++k) { h->Wss[k] = wp(o_wss[k]); h->Wg[k] = wp(o_wg[k]); h->W1[k] = wp(o_w1[k]); h->W2[k] = wp(o_w2[k]); }

  // ---- fp32 side parameters
  std::vector<float> fs;
  auto put = [&](const float* src, size_t n) { size_t o = fs.size(); fs.insert(fs.end(), src, src + n); while (fs.size() % 4) fs.push_back(0.0f); return o; };
  const size_t f_bz = put(w->bz, W), f_wt1 = put(w->Wt1, W * F), f_bt1 = put(w->bt1, W), f_wt2 = put(w->Wt2, W * W),
               f_bt2 = put(w->bt2, W), f_bin = put(w->bin, W);
  // Wout transposed to [W, 16] (or [W, 32] for a head that also predicts its variances: columns 16.. hold the
  // variance rows C..2C of Wout), zero padded; the eps columns sit where they sit in a fixed-variance head
  const size_t epw = d.var_out ? kCPad2 : kCPad;
  std::vector<float> win_pad(W * kCPad, 0.0f), wout_t(W * epw, 0.0f), bout_pad(epw, 0.0f);
  for (size_t n = 0; n < W; ++n)
    for (size_t c = 0; c < C; ++c) {
      win_pad[n * kCPad + c] = w->Win[n * C + c];
      wout_t[n * epw + c] = w->Wout[c * W + n];
      if (d.var_out) wout_t[n * epw + kCPad + c] = w->Wout[(C + c) * W + n];
    }
  for (size_t c = 0; c < C; ++c) { bout_pad[c] = w->bout[c]; if (d.var_out) bout_pad[kCPad + c] = w->bout[C + c]; }
  const size_t f_win = put(win_pad.data(), win_pad.size()), f_wout = put(wout_t.data(), wout_t.size()),
               f_bout = put(bout_pad.data(), epw);
  std::vector<size_t> f_bsh(L), f_bsc(L), f_bg(L), f_b1(L), f_b2(L);
  for (size_t k = 0; k < L; ++k) {
    f_bsh[k] = put(w->bada + k * 3 * W, W); f_bsc[k] = put(w->bada + k * 3 * W + W, W);
    f_bg[k] = put(w->bada + k * 3 * W + 2 * W, W);
    f_b1[k] = put(w->b1 + k * W, W); f_b2[k] = put(w->b2 + k * W, W);
  }
  const size_t f_bfsh = put(w->bfada, W), f_bfsc = put(w->bfada + W, W);
  // folded blocks: c1_k = W1_k (1 + bscale_k), c2_k = W1_k bshift_k + b1_k  (double accumulation, rounded once)
  const bool folded = d.dtype != CSD_F32 && L >= 2;
  // the small-batch chain kernel folds every block, the first included
  const bool sbk = d.dtype != CSD_F32 && W % 512 == 0 && W <= static_cast<size_t>(kSbMaxW) && !d.var_out;
  const size_t kfold0 = sbk ? 0 : 1;      // first block that has folded weights
  std::vector<size_t> f_c1(L, 0), f_c2(L, 0);
  if (folded || sbk) {
    std::vector<float> v1(W), v2(W);
    for (size_t k = kfold0; k < L; ++k) {
      const float* W1k = w->W1 + k * W * W;
      const float* bsh = w->bada + k * 3 * W;
      const float* bsc = bsh + W;
      for (size_t n = 0; n < W; ++n) {
        double a1 = 0.0, a2 = 0.0;
        for (size_t j = 0; j < W; ++j) { a1 += static_cast<double>(W1k[n * W + j]) * (1.0 + bsc[j]); a2 += static_cast<double>(W1k[n * W + j]) * bsh[j]; }
        v1[n] = static_cast<float>(a1); v2[n] = static_cast<float>(a2 + w->b1[k * W + n]);
      }
      f_c1[k] = put(v1.data(), W); f_c2[k] = put(v2.data(), W);
    }
  }
  if (cudaMalloc(&h->fblob, fs.size() * 4) != cudaSuccess) { cudaGetLastError(); return bail(CSD_ERR_WORKSPACE, "cannot allocate device memory for the parameters"); }
  if (cudaMemcpy(h->fblob, fs.data(), fs.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess) return bail(CSD_ERR_CUDA, "parameter upload failed");
  float* fb = h->fblob;
  h->bz = fb + f_bz; h->Wt1 = fb + f_wt1; h->bt1 = fb + f_bt1; h->Wt2 = fb + f_wt2; h->bt2 = fb + f_bt2;
  h->win = fb + f_win; h->bin = fb + f_bin; h->wout_t = fb + f_wout; h->bout = fb + f_bout;
  h->bfsh = fb + f_bfsh; h->bfsc = fb + f_bfsc;
  h->c1.assign(L, nullptr); h->c2.assign(L, nullptr);
  if (folded || sbk) for (size_t k = kfold0; k < L; ++k) { h->c1[k] = fb + f_c1[k]; h->c2[k] = fb + f_c2[k]; }
  h->bsh.resize(L); h->bsc.resize(L); h->bg.resize(L); h->b1.resize(L); h->b2.resize(L);
  for (size_t k = 0; k < L; ++k) { h->bsh[k] = fb + f_bsh[k]; h->bsc[k] = fb + f_bsc[k]; h->bg[k] = fb + f_bg[k]; h->b1[k] = fb + f_b1[k]; h->b2[k] = fb + f_b2[k]; }

  if (d.dtype != CSD_F32) {
    int rc = CSD_OK;
    for (int i = 0; i < 2 && !rc; ++i) {
      const uint32_t tn = i == 0 ? 64 : 128;   // B box rows = MMA N: tn, or 2 tn for the interleaved shift | scale rows
      csd_head::TmSet& tm = h->tm[i];
      rc = make_tmap(ctx, &tm.Wz, d.dtype, h->Wz, W, Dz, Dz, tn);
      tm.Wss.resize(L); tm.Wg.resize(L); tm.W1.resize(L); tm.W2.resize(L);
      for (size_t k = 0; k < L && !rc; ++k) {
        rc = make_tmap(ctx, &tm.Wss[k], d.dtype, h->Wss[k], 2 * W, W, W, 2 * tn);
        if (!rc) rc = make_tmap(ctx, &tm.Wg[k], d.dtype, h->Wg[k], W, W, W, tn);
        if (!rc) rc = make_tmap(ctx, &tm.W1[k], d.dtype, h->W1[k], W, W, W, tn);
        if (!rc) rc = make_tmap(ctx, &tm.W2[k], d.dtype, h->W2[k], W, W, W, tn);
      }
      if (!rc) rc = make_tmap(ctx, &tm.Wfss, d.dtype, h->Wfss, 2 * W, W, W, 2 * tn);
    }
    std::vector<CUtensorMap> wf128(L);
    if (!rc && (folded || sbk)) {
      // xblob: Wgs_0 .. Wgs_{L-2} | Wf_1 .. Wf_{L-1} | Wf_0 (small-batch kernel only), each [2 W, W] in operand format
      const size_t per = 2 * W * W, nx = (2 * (L - 1) + (sbk ? 1 : 0)) * per;
      auto wf_slot = [&](size_t k) { return k == 0 ? 2 * (L - 1) : L - 1 + k - 1; };
      std::vector<float> xs;
      try { xs.resize(nx); } catch (...) { return bail(CSD_ERR_WORKSPACE, "out of host memory"); }
      float *dA = nullptr, *dB = nullptr, *dC = nullptr;
      std::vector<float> f1(W * W), f2(W * W);
      bool okx = cudaMalloc(&dA, W * W * 4) == cudaSuccess && cudaMalloc(&dB, W * W * 4) == cudaSuccess && cudaMalloc(&dC, W * W * 4) == cudaSuccess;
      for (size_t k = 0; k + 1 < L && okx; ++k)     // gate of block k | scale of block k + 1
        interleave(w->Wada + k * 3 * W * W + 2 * W * W, w->Wada + (k + 1) * 3 * W * W + W * W, &xs[k * per]);
      for (size_t k = kfold0; k < L && okx; ++k) {  // W1_k Wscale_k | W1_k Wshift_k
        const float* ada = w->Wada + k * 3 * W * W;
        const dim3 grid(static_cast<unsigned>(W / 32), static_cast<unsigned>(W / 32));
        okx = okx && cudaMemcpy(dA, w->W1 + k * W * W, W * W * 4, cudaMemcpyHostToDevice) == cudaSuccess;
        okx = okx && cudaMemcpy(dB, ada + W * W, W * W * 4, cudaMemcpyHostToDevice) == cudaSuccess;
        if (okx) square_matmul_kernel<<<grid, 256>>>(dA, dB, dC, static_cast<int>(W));
        okx = okx && cudaMemcpy(f1.data(), dC, W * W * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
        okx = okx && cudaMemcpy(dB, ada, W * W * 4, cudaMemcpyHostToDevice) == cudaSuccess;
        if (okx) square_matmul_kernel<<<grid, 256>>>(dA, dB, dC, static_cast<int>(W));
        okx = okx && cudaMemcpy(f2.data(), dC, W * W * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
        if (okx) interleave(f1.data(), f2.data(), &xs[wf_slot(k) * per]);
      }
      if (dA) cudaFree(dA);
      if (dB) cudaFree(dB);
      if (dC) cudaFree(dC);
      if (!okx) { cudaGetLastError(); return bail(CSD_ERR_CUDA, "fused weight products failed"); }
      std::vector<uint16_t> xb;
      try { xb.resize(nx); } catch (...) { return bail(CSD_ERR_WORKSPACE, "out of host memory"); }
      if (d.dtype == CSD_BF16) { for (size_t i = 0; i < nx; ++i) xb[i] = f32_to_bf16_bits(xs[i]); }
      else { for (size_t i = 0; i < nx; ++i) { const __half hv = __float2half_rn(xs[i]); memcpy(&xb[i], &hv, 2); } }
      if (cudaMalloc(&h->xblob, nx * 2) != cudaSuccess) { cudaGetLastError(); return bail(CSD_ERR_WORKSPACE, "cannot allocate device memory for the fused weights"); }
      if (cudaMemcpy(h->xblob, xb.data(), nx * 2, cudaMemcpyHostToDevice) != cudaSuccess) return bail(CSD_ERR_CUDA, "fused weight upload failed");
      h->Wgs.resize(L); h->Wf.resize(L); h->Wgs_half.resize(L); h->Wf_half.resize(L);
      char* xbase = static_cast<char*>(h->xblob);
      for (size_t k = 0; k + 1 < L && !rc; ++k) rc = make_tmap(ctx, &h->Wgs[k], d.dtype, xbase + k * per * 2, 2 * W, W, W, 256);
      for (size_t k = 1; k < L && !rc; ++k) rc = make_tmap(ctx, &h->Wf[k], d.dtype, xbase + wf_slot(k) * per * 2, 2 * W, W, W, 256);
      for (size_t k = 0; k + 1 < L && !rc; ++k) rc = make_tmap(ctx, &h->Wgs_half[k], d.dtype, xbase + k * per * 2, 2 * W, W, W, 128);
      for (size_t k = kfold0; k < L && !rc; ++k) rc = make_tmap(ctx, &h->Wf_half[k], d.dtype, xbase + wf_slot(k) * per * 2, 2 * W, W, W, 128);
      for (size_t k = kfold0; k < L && !rc && sbk; ++k) rc = make_tmap(ctx, &wf128[k], d.dtype, xbase + wf_slot(k) * per * 2, 2 * W, W, W, 128);
    }
    if (!rc && W % 256 == 0) {
      h->W1_wide.resize(L);
      for (size_t k = 0; k < L && !rc; ++k) rc = make_tmap(ctx, &h->W1_wide[k], d.dtype, h->W1[k], W, W, W, 256);
    }
    if (rc) { csd_head_destroy(h); return rc; }
    if (sbk) {
      // tables of the small-batch chain kernel
      std::vector<CUtensorMap> maps;
      for (size_t k = 0; k < L; ++k) { maps.push_back(h->tm[1].W1[k]); maps.push_back(h->tm[1].W2[k]); }
      std::vector<SbTask> tasks;
      auto add = [&](const CUtensorMap& m, size_t rows, size_t col0) {
        const int mi = static_cast<int>(maps.size());
        maps.push_back(m);
        for (size_t r = 0; r < rows; r += 128) tasks.push_back(SbTask{mi, static_cast<int>(r), static_cast<int>(col0 + r), 0});
      };
      for (size_t k = 0; k < L; ++k) {           // mods columns of block k: [P1 | P2 : 2 W][gate : W][shift | scale : 2 W]
        add(wf128[k], 2 * W, 5 * k * W);
        add(h->tm[1].Wg[k], W, 5 * k * W + 2 * W);
        add(h->tm[0].Wss[k], 2 * W, 5 * k * W + 3 * W);
      }
      add(h->tm[0].Wfss, 2 * W, 5 * L * W);
      std::vector<const float*> bt;
      for (size_t k = 0; k < L; ++k) { bt.push_back(h->c1[k]); bt.push_back(h->c2[k]); bt.push_back(h->bg[k]); bt.push_back(h->b2[k]); bt.push_back(h->bsc[k]); }
      bt.push_back(h->bfsh); bt.push_back(h->bfsc);
      if (cudaMalloc(&h->d_sb_maps, maps.size() * sizeof(CUtensorMap)) != cudaSuccess ||
          cudaMalloc(&h->d_sb_tasks, tasks.size() * sizeof(SbTask)) != cudaSuccess ||
          cudaMalloc(&h->d_sb_bias, bt.size() * sizeof(float*)) != cudaSuccess) { cudaGetLastError(); return bail(CSD_ERR_WORKSPACE, "cannot allocate device memory for the small-batch tables"); }
      if (cudaMemcpy(h->d_sb_maps, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice) != cudaSuccess ||
          cudaMemcpy(h->d_sb_tasks, tasks.data(), tasks.size() * sizeof(SbTask), cudaMemcpyHostToDevice) != cudaSuccess ||
          cudaMemcpy(h->d_sb_bias, bt.data(), bt.size() * sizeof(float*), cudaMemcpyHostToDevice) != cudaSuccess) return bail(CSD_ERR_CUDA, "small-batch table upload failed");
      h->sb_ntasks = static_cast<int>(tasks.size());
      h->sb_ready = true;
    }
    if (sbk && W / kTileN == static_cast<size_t>(kPcColTiles)) {
      // tables of the persistent chain kernel: phases B, (W1_k, GATE_k) for every block, F
      const size_t NP = 2 * L + 2;
      std::vector<CUtensorMap> maps(2 * NP);
      std::vector<const float*> bt(3 * NP, nullptr);
      maps[0] = h->tm[0].Wss[0]; bt[0] = h->bsc[0];
      for (size_t k = 0; k < L; ++k) {
        const size_t w1 = 1 + 2 * k, gt = 2 + 2 * k;
        maps[w1] = h->Wf_half[k]; maps[NP + w1] = h->tm[0].W1[k]; bt[3 * w1] = h->c1[k]; bt[3 * w1 + 1] = h->c2[k];
        maps[gt] = k + 1 < L ? h->Wgs_half[k] : h->tm[0].Wg[k]; maps[NP + gt] = h->tm[0].W2[k];
        bt[3 * gt] = h->bg[k]; bt[3 * gt + 1] = h->b2[k]; bt[3 * gt + 2] = k + 1 < L ? h->bsc[k + 1] : nullptr;
      }
      maps[NP - 1] = h->tm[0].Wfss; bt[3 * (NP - 1)] = h->bfsh; bt[3 * (NP - 1) + 1] = h->bfsc;
      maps[NP] = h->tm[0].W1[0]; maps[2 * NP - 1] = h->tm[0].W1[0];   // unused entries: any valid map
      if (cudaMalloc(&h->d_pc_maps, maps.size() * sizeof(CUtensorMap)) != cudaSuccess ||
          cudaMalloc(&h->d_pc_bias, bt.size() * sizeof(float*)) != cudaSuccess) { cudaGetLastError(); return bail(CSD_ERR_WORKSPACE, "cannot allocate device memory for the persistent-chain tables"); }
      if (cudaMemcpy(h->d_pc_maps, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice) != cudaSuccess ||
          cudaMemcpy(h->d_pc_bias, bt.data(), bt.size() * sizeof(float*), cudaMemcpyHostToDevice) != cudaSuccess) return bail(CSD_ERR_CUDA, "persistent-chain table upload failed");
      h->pc_ready = true;
    }
  }
  *out = h;
  return CSD_OK;
}

int csd_head_destroy(csd_head* h) {
  if (!h) return CSD_ERR_INVALID_ARG;
  DeviceGuard dg(h->ctx ? h->ctx->device : 0);
  if (h->ctx) {
    cudaStreamSynchronize(h->ctx->stream);
    for (int i = 0; i < 2; ++i) cudaStreamSynchronize(h->ctx->side[i]);
  }
  if (h->wblob) cudaFree(h->wblob);
  if (h->fblob) cudaFree(h->fblob);
  if (h->xblob) cudaFree(h->xblob);
  if (h->d_pc_maps) cudaFree(h->d_pc_maps);
  if (h->d_pc_bias) cudaFree(h->d_pc_bias);
  if (h->d_sb_maps) cudaFree(h->d_sb_maps);
  if (h->d_sb_tasks) cudaFree(h->d_sb_tasks);
  if (h->d_sb_bias) cudaFree(h->d_sb_bias);
  cudaGetLastError();
  delete h;
  return CSD_OK;
}

int csd_draft_denoise(csd_ctx* ctx, const csd_head* head, const csd_schedule* sched, int R, int cfg, float cfg_scale,
                      const float* z, const float* x_T, const float* eps, float* x0, float* mu1, float* x1) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  int rc = check_chain_args(ctx, head, sched, R, cfg, z, x_T, eps);
  if (rc) return rc;
  if (!x0 || !mu1) return fail(ctx, CSD_ERR_INVALID_ARG, "x0 / mu1 is null");
  CSD_DEVICE(ctx);
  return run_chain(ctx, 0, ctx->stream, head, sched, R, cfg, cfg_scale, z, x_T, eps, 1, x0, mu1, x1);
}

// ---------------------------------------------------------------------------------------------
// csd_draft_denoise_static: the same kernels as csd_draft_denoise, but every intermediate buffer
// lives in this one file-scope device array instead of a cudaMalloc'ed workspace.
constexpr size_t kStaticScratchBytes = size_t(8) << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
static void* g_static_scratch_addr[kMaxDevices] = {nullptr};   // device address of the array, per device ordinal

int csd_draft_denoise_static(csd_ctx* ctx, const csd_head* head, const csd_schedule* sched, int R, int cfg,
                             float cfg_scale, const float* z, const float* x_T, const float* eps, float* x0,
                             float* mu1, float* x1) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  int rc = check_chain_args(ctx, head, sched, R, cfg, z, x_T, eps);
  if (rc) return rc;
  if (!x0 || !mu1) return fail(ctx, CSD_ERR_INVALID_ARG, "x0 / mu1 is null");
  if (ctx->prof_on) return fail(ctx, CSD_ERR_INVALID_ARG, "csd_draft_denoise_static: switch csd_profile off first (recording creates CUDA events)");
  CSD_DEVICE(ctx);
  // Bytes the chain's intermediates need: the same layout function the growable workspaces use.  Reject before
  // anything is enqueued.
  const csd_head_desc& d = head->d;
  const size_t need = ws_layout(d, R * (cfg ? 2 : 1), R, sched->T).total;
  if (need > kStaticScratchBytes)
    return fail(ctx, CSD_ERR_WORKSPACE,
                "csd_draft_denoise_static: this call needs %zu bytes of scratch but the built-in array holds %zu "
                "(rows R=%d%s, width %d, T=%d); use csd_draft_denoise or fewer rows", need, kStaticScratchBytes, R,
                cfg ? " doubled by guidance" : "", d.W, sched->T);
  // First call on this device: look up the device address of the array (the symbol's name is only a
  // host-side stand-in and must never be handed to a kernel).
  if (!g_static_scratch_addr[ctx->device]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) {
      cudaGetLastError();
      return fail(ctx, CSD_ERR_CUDA, "cudaGetSymbolAddress(static scratch) failed: %s", cudaGetErrorString(e));
    }
    g_static_scratch_addr[ctx->device] = p;
  }
  ChainWs& ws = ctx->ws[2];
  ws.base = g_static_scratch_addr[ctx->device];
  ws.cap = kStaticScratchBytes;
  ws.owned = false;                      // never freed or grown: a call that does not fit is an error
  return run_chain(ctx, 2, ctx->stream, head, sched, R, cfg, cfg_scale, z, x_T, eps, 1, x0, mu1, x1);
}

int csd_accept_scan(csd_ctx* ctx, int B, int gamma, int C, double log_sigma_term_, float sigma1_p, float sigma1_q,
                    const float* x0_q, const float* mu1_q, const float* mu1_p, const float* u, float* logratio,
                    int32_t* n_accept, uint32_t* accept_mask) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  int rc = check_verify_dims(ctx, B, gamma, C);
  if (rc) return rc;
  if (!x0_q || !mu1_q || !mu1_p || !u || !logratio || !n_accept) return fail(ctx, CSD_ERR_INVALID_ARG, "null array argument");
  if (!(sigma1_p > 0.0f) || !(sigma1_q > 0.0f)) return fail(ctx, CSD_ERR_INVALID_ARG, "sigma1 must be > 0");
  CSD_DEVICE(ctx);
  return accept_scan(ctx, ctx->stream, B, gamma, C, log_sigma_term_, sigma1_p, sigma1_q, x0_q, mu1_q, mu1_p, u, logratio,
                     n_accept, accept_mask);
}

static int verify_impl(csd_ctx* ctx, const csd_head* head_p, const csd_schedule* sched_p, const csd_schedule* sched_q,
                       int B, int gamma, int cfg, float cfg_scale, const float* z_p, const float* x_T, const float* eps,
                       const float* x0_q, const float* mu1_q, const float* u, float* logratio, int32_t* n_accept,
                       uint32_t* accept_mask, float* mu1_p, bool bonus, const float* z_next, const float* x_T_next,
                       const float* eps_next, float* x_bonus, uint32_t* taken) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  if (B < 1 || gamma < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "B = %d and gamma = %d must be >= 1", B, gamma);
  int rc = check_chain_args(ctx, head_p, sched_p, B * gamma, cfg, z_p, x_T, eps);
  if (rc) return rc;
  if ((rc = check_sched(ctx, sched_q, false))) return rc;
  if (sched_q->T != sched_p->T) return fail(ctx, CSD_ERR_SHAPE, "draft T = %d and target T = %d differ", sched_q->T, sched_p->T);
  if ((rc = check_verify_dims(ctx, B, gamma, head_p->d.C))) return rc;
  if (!x0_q || !mu1_q || !u || !logratio || !n_accept || !mu1_p) return fail(ctx, CSD_ERR_INVALID_ARG, "null array argument");
  if (bonus && (!z_next || !x_T_next || !eps_next || !x_bonus)) return fail(ctx, CSD_ERR_INVALID_ARG, "z_next / x_T_next / eps_next / x_bonus is null");
  CSD_DEVICE(ctx);
  const int R = B * gamma, C = head_p->d.C, T = sched_p->T;
  BonusBuf bb{};
  if (bonus) {
    if ((rc = ensure_side(ctx, ctx->bn, bonus_buf_bytes(head_p->d, R + B, cfg, T), "the bonus rows"))) return rc;
    if ((rc = gather_bonus_inputs(ctx, ctx->stream, head_p->d, R, B, cfg, T, z_p, x_T, eps, z_next, x_T_next, eps_next, bb))) return rc;
    // every row samples at the last step; only the bonus rows' samples are used
    rc = run_chain(ctx, 1, ctx->stream, head_p, sched_p, R + B, cfg, cfg_scale, bb.z, bb.x_T, bb.eps, 1, bb.x0, bb.mu1, nullptr);
    if (rc) return rc;
    CSD_CUDA(ctx, cudaMemcpyAsync(mu1_p, bb.mu1, static_cast<size_t>(R) * C * 4, cudaMemcpyDeviceToDevice, ctx->stream));
  } else {
    rc = run_chain(ctx, 1, ctx->stream, head_p, sched_p, R, cfg, cfg_scale, z_p, x_T, eps, 0, nullptr, mu1_p, nullptr);
    if (rc) return rc;
  }
  rc = accept_scan(ctx, ctx->stream, B, gamma, C, log_sigma_term(sched_q, sched_p, C), sched_p->sigma[0],
                   sched_q->sigma[0], x0_q, mu1_q, mu1_p, u, logratio, n_accept, accept_mask);
  if (rc || !bonus) return rc;
  bonus_select_kernel<<<(B * C + 255) / 256, 256, 0, ctx->stream>>>(B, C, gamma, n_accept, bb.x0 + static_cast<size_t>(R) * C, x_bonus, taken);
  ctx->launches++;
  CSD_CUDA(ctx, cudaGetLastError());
  return CSD_OK;
}

int csd_verify(csd_ctx* ctx, const csd_head* head_p, const csd_schedule* sched_p, const csd_schedule* sched_q, int B,
               int gamma, int cfg, float cfg_scale, const float* z_p, const float* x_T, const float* eps,
               const float* x0_q, const float* mu1_q, const float* u, float* logratio, int32_t* n_accept,
               uint32_t* accept_mask, float* mu1_p) {
  return verify_impl(ctx, head_p, sched_p, sched_q, B, gamma, cfg, cfg_scale, z_p, x_T, eps, x0_q, mu1_q, u, logratio,
                     n_accept, accept_mask, mu1_p, false, nullptr, nullptr, nullptr, nullptr, nullptr);
}

int csd_verify_bonus(csd_ctx* ctx, const csd_head* head_p, const csd_schedule* sched_p, const csd_schedule* sched_q, int B,
                     int gamma, int cfg, float cfg_scale, const float* z_p, const float* x_T, const float* eps,
                     const float* x0_q, const float* mu1_q, const float* u, const float* z_next, const float* x_T_next,
                     const float* eps_next, float* logratio, int32_t* n_accept, uint32_t* accept_mask, float* mu1_p,
                     float* x_bonus, uint32_t* taken) {
  return verify_impl(ctx, head_p, sched_p, sched_q, B, gamma, cfg, cfg_scale, z_p, x_T, eps, x0_q, mu1_q, u, logratio,
                     n_accept, accept_mask, mu1_p, true, z_next, x_T_next, eps_next, x_bonus, taken);
}

int csd_verify_unaligned(csd_ctx* ctx, const csd_head* head_p, const csd_schedule* sched_p, const csd_schedule* sched_q,
                         int B, int gamma, int cfg, float cfg_scale, const float* z_p, const float* x_T,
                         const float* eps_p, const float* eps_q, const float* x0_q, const float* mu1_q, const float* u,
                         float* logratio, int32_t* n_accept, uint32_t* accept_mask, float* mu1_p) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  if (B < 1 || gamma < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "B = %d and gamma = %d must be >= 1", B, gamma);
  int rc = check_chain_args(ctx, head_p, sched_p, B * gamma, cfg, z_p, x_T, eps_p);
  if (rc) return rc;
  if ((rc = check_sched(ctx, sched_q, false))) return rc;
  if (sched_q->T != sched_p->T) return fail(ctx, CSD_ERR_SHAPE, "draft T = %d and target T = %d differ", sched_q->T, sched_p->T);
  if ((rc = check_verify_dims(ctx, B, gamma, head_p->d.C))) return rc;
  if (!eps_q || !x0_q || !mu1_q || !u || !logratio || !n_accept || !mu1_p) return fail(ctx, CSD_ERR_INVALID_ARG, "null array argument");
  CSD_DEVICE(ctx);
  const int R = B * gamma, C = head_p->d.C, T = sched_p->T;
  const size_t need = static_cast<size_t>(R) * 4;
  if (need > ctx->un.cap) {
    CSD_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (ctx->un.base) CSD_CUDA(ctx, cudaFree(ctx->un.base));
    ctx->un.base = nullptr; ctx->un.cap = 0;
    if (cudaMalloc(&ctx->un.base, need) != cudaSuccess) {
      cudaGetLastError();
      return fail(ctx, CSD_ERR_WORKSPACE, "cannot allocate %zu bytes for the noise terms", need);
    }
    ctx->un.cap = need;
  }
  float* d_off = static_cast<float*>(ctx->un.base);
  rc = run_chain(ctx, 1, ctx->stream, head_p, sched_p, R, cfg, cfg_scale, z_p, x_T, eps_p, 0, nullptr, mu1_p, nullptr);
  if (rc) return rc;
  noise_norm_term_kernel<<<(R + 127) / 128, 128, 0, ctx->stream>>>(R, C, T, eps_q, eps_p, d_off);
  ctx->launches++;
  CSD_CUDA(ctx, cudaGetLastError());
  return accept_scan(ctx, ctx->stream, B, gamma, C, log_sigma_term(sched_q, sched_p, C), sched_p->sigma[0],
                     sched_q->sigma[0], x0_q, mu1_q, mu1_p, u, logratio, n_accept, accept_mask, d_off);
}

int csd_bonus_token(csd_ctx* ctx, const csd_head* head_p, const csd_schedule* sched_p, int B, int gamma, int cfg,
                    float cfg_scale, const float* z_next, const float* x_T_next, const float* eps_next,
                    const int32_t* n_accept, float* x_bonus, uint32_t* taken) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  if (gamma < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "gamma = %d must be >= 1", gamma);
  int rc = check_chain_args(ctx, head_p, sched_p, B, cfg, z_next, x_T_next, eps_next);
  if (rc) return rc;
  if (!n_accept || !x_bonus) return fail(ctx, CSD_ERR_INVALID_ARG, "n_accept / x_bonus is null");
  CSD_DEVICE(ctx);
  const int C = head_p->d.C;
  if ((rc = ensure_side(ctx, ctx->bn, static_cast<size_t>(2) * B * C * 4, "the bonus samples"))) return rc;
  float* d_x0 = static_cast<float*>(ctx->bn.base);
  float* d_mu = d_x0 + static_cast<size_t>(B) * C;
  // the masks live on the device, so every sequence is sampled and the selection is a kernel: no host round trip
  rc = run_chain(ctx, 1, ctx->stream, head_p, sched_p, B, cfg, cfg_scale, z_next, x_T_next, eps_next, 1, d_x0, d_mu, nullptr);
  if (rc) return rc;
  bonus_select_kernel<<<(B * C + 255) / 256, 256, 0, ctx->stream>>>(B, C, gamma, n_accept, d_x0, x_bonus, taken);
  ctx->launches++;
  CSD_CUDA(ctx, cudaGetLastError());
  return CSD_OK;
}

int csd_draft_denoise_traj(csd_ctx* ctx, const csd_head* head, const csd_schedule* sched, int R, int cfg,
                           float cfg_scale, const float* z, const float* x_T, const float* eps, float* traj_x,
                           float* traj_mu) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  int rc = check_chain_args(ctx, head, sched, R, cfg, z, x_T, eps);
  if (rc) return rc;
  if (!traj_x || !traj_mu) return fail(ctx, CSD_ERR_INVALID_ARG, "traj_x / traj_mu is null");
  CSD_DEVICE(ctx);
  const size_t slot = static_cast<size_t>(R) * head->d.C;
  const int T = sched->T;
  // the last boundary writes x_0 and mu_1 through the chain's ordinary outputs, which are the last slots
  Chain c{ctx, 0, ctx->stream, head, sched, R, cfg, cfg_scale, z, x_T, eps, 1, traj_x + T * slot,
          traj_mu + (T - 1) * slot, nullptr};
  c.traj_x = traj_x; c.traj_mu = traj_mu;
  rc = c.begin();
  for (int t = T; t >= 1 && !rc; --t) rc = c.step(t);
  return rc;
}

int csd_verify_single_path(csd_ctx* ctx, const csd_head* head_p, const csd_schedule* sched_p,
                           const csd_schedule* sched_q, int B, int gamma, int cfg, float cfg_scale, const float* z_p,
                           const float* traj_x, const float* traj_mu_q, const float* u, int steps_per_pass,
                           float* logratio, int32_t* n_accept, uint32_t* accept_mask, float* mu_p_traj) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  if (B < 1 || gamma < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "B = %d and gamma = %d must be >= 1", B, gamma);
  if (static_cast<int64_t>(B) * gamma > (1 << 24)) return fail(ctx, CSD_ERR_UNSUPPORTED, "B * gamma exceeds 2^24 rows");
  const int R = B * gamma;
  if (!traj_x || !traj_mu_q) return fail(ctx, CSD_ERR_INVALID_ARG, "traj_x / traj_mu_q is null");
  int rc = check_chain_args(ctx, head_p, sched_p, R, cfg, z_p, traj_x, traj_mu_q);
  if (rc) return rc;
  if ((rc = check_sched(ctx, sched_q, false))) return rc;
  if (sched_q->T != sched_p->T) return fail(ctx, CSD_ERR_SHAPE, "draft T = %d and target T = %d differ", sched_q->T, sched_p->T);
  if ((rc = check_verify_dims(ctx, B, gamma, head_p->d.C))) return rc;
  if (!u || !logratio || !n_accept) return fail(ctx, CSD_ERR_INVALID_ARG, "null array argument");
  if (steps_per_pass < 0) return fail(ctx, CSD_ERR_INVALID_ARG, "steps_per_pass = %d must be >= 0", steps_per_pass);
  CSD_DEVICE(ctx);
  const int T = sched_p->T, C = head_p->d.C, Rh1 = R * (cfg ? 2 : 1);
  // steps per pass: enough head rows to fill the GPU several times over, few enough to keep the workspace
  // (about 16 W bytes per head row) modest
  constexpr int kRowsPerPass = 32768;
  int tb = steps_per_pass ? steps_per_pass : (kRowsPerPass + Rh1 - 1) / Rh1;
  if (tb > T) tb = T;
  if (static_cast<int64_t>(tb) * Rh1 > (int64_t(1) << 26)) return fail(ctx, CSD_ERR_UNSUPPORTED, "pass of %d steps has too many rows", tb);
  // device side buffer: [5, T] constants | mu^p of a pass [tb R, C] | per-step terms [T, R]
  const size_t o_mu = align_up(static_cast<size_t>(5) * T * 4, 256);
  const size_t o_acc = align_up(o_mu + static_cast<size_t>(tb) * R * C * 4, 256);
  const size_t need = o_acc + static_cast<size_t>(T) * R * 4;
  cudaStream_t st = ctx->stream;
  if (need > ctx->sp.cap) {
    CSD_CUDA(ctx, cudaStreamSynchronize(st));
    if (ctx->sp.base) CSD_CUDA(ctx, cudaFree(ctx->sp.base));
    ctx->sp.base = nullptr; ctx->sp.cap = 0;
    if (cudaMalloc(&ctx->sp.base, need) != cudaSuccess) {
      cudaGetLastError();
      return fail(ctx, CSD_ERR_WORKSPACE, "cannot allocate %zu bytes for the single-path buffers", need);
    }
    ctx->sp.cap = need;
  }
  char* base = static_cast<char*>(ctx->sp.base);
  float* d_sched = reinterpret_cast<float*>(base);
  float* d_mu = reinterpret_cast<float*>(base + o_mu);
  float* d_terms = reinterpret_cast<float*>(base + o_acc);
  {
    // per step: a_t, b_t of the target, C (log sigma_q,t - log sigma_p,t), 1 / (2 sigma_p,t^2), 1 / (2 sigma_q,t^2)
    std::vector<float> hs(static_cast<size_t>(5) * T);
    for (int t = 0; t < T; ++t) {
      const double sp = sched_p->sigma[t], sq = sched_q->sigma[t];
      hs[t] = sched_p->a[t]; hs[T + t] = sched_p->b[t];
      hs[2 * T + t] = static_cast<float>(C * (std::log(sq) - std::log(sp)));
      hs[3 * T + t] = static_cast<float>(0.5 / (sp * sp));
      hs[4 * T + t] = static_cast<float>(0.5 / (sq * sq));
    }
    // pageable source: the runtime stages it before the call returns
    CSD_CUDA(ctx, cudaMemcpyAsync(d_sched, hs.data(), hs.size() * 4, cudaMemcpyHostToDevice, st));
  }
  for (int j0 = 0; j0 < T; j0 += tb) {
    const int n = T - j0 < tb ? T - j0 : tb;
    Chain c{ctx, 1, st, head_p, sched_p, n * R, cfg, cfg_scale, z_p, nullptr, nullptr, 0, nullptr, nullptr, nullptr};
    // the target's means of this pass: into the caller's [T, R, C] array (slot j0 onwards) when it wants them
    float* pass_mu = mu_p_traj ? mu_p_traj + static_cast<size_t>(j0) * R * C : d_mu;
    c.batch_Rin = R; c.batch_j0 = j0; c.batch_traj = traj_x; c.batch_sched = d_sched; c.batch_mu = pass_mu;
    c.ws_steps = tb; c.batch_reuse = j0 > 0;
    if ((rc = c.begin())) return rc;
    if ((rc = c.step(1))) return rc;
    single_path_terms_kernel<<<(n * R + 127) / 128, 128, 0, st>>>(R, C, T, j0, n, d_sched, traj_x, traj_mu_q, pass_mu, d_terms);
    ctx->launches++;
    CSD_CUDA(ctx, cudaGetLastError());
  }
  single_path_accept_kernel<<<(B + 3) / 4, 128, 0, st>>>(B, gamma, T, d_terms, u, logratio, n_accept, accept_mask);
  ctx->launches++;
  CSD_CUDA(ctx, cudaGetLastError());
  return CSD_OK;
}

int csd_resample(csd_ctx* ctx, int B, int gamma, int C, int cap, double log_sigma_term_, float sigma1_p, float sigma1_q,
                 const int32_t* n_accept, const float* mu1_p, const float* mu1_q, const float* xi, const float* v,
                 float* x_new, int32_t* n_prop, uint32_t* flags, int32_t* cap_hits) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  int rc = check_verify_dims(ctx, B, gamma, C);
  if (rc) return rc;
  if (cap < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "cap = %d must be >= 1", cap);
  if (!n_accept || !mu1_p || !mu1_q || !xi || !v || !x_new || !n_prop || !flags || !cap_hits)
    return fail(ctx, CSD_ERR_INVALID_ARG, "null array argument");
  if (!(sigma1_p > 0.0f) || !(sigma1_q > 0.0f)) return fail(ctx, CSD_ERR_INVALID_ARG, "sigma1 must be > 0");
  CSD_DEVICE(ctx);
  return resample(ctx, ctx->stream, B, gamma, C, cap, log_sigma_term_, sigma1_p, sigma1_q, n_accept, mu1_p, mu1_q, xi, v,
                  x_new, n_prop, flags, cap_hits);
}

static int round_impl(csd_ctx* ctx, const csd_head* head_q, const csd_head* head_p, const csd_schedule* sched_q,
                      const csd_schedule* sched_p, int B, int gamma, int cfg, float cfg_scale, int cap, const float* z_q,
                      const float* z_p, const float* x_T, const float* eps, const float* u, const float* xi,
                      const float* v, float* x0, float* mu1_q, float* mu1_p, float* logratio, int32_t* n_accept,
                      uint32_t* accept_mask, float* x_new, int32_t* n_prop, uint32_t* flags, int32_t* cap_hits,
                      bool bonus, const float* z_next, const float* x_T_next, const float* eps_next, float* x_bonus,
                      uint32_t* taken) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  if (B < 1 || gamma < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "B = %d and gamma = %d must be >= 1", B, gamma);
  const int R = B * gamma;
  int rc = check_chain_args(ctx, head_q, sched_q, R, cfg, z_q, x_T, eps);
  if (rc) return rc;
  if ((rc = check_chain_args(ctx, head_p, sched_p, R, cfg, z_p, x_T, eps))) return rc;
  if (sched_q->T != sched_p->T) return fail(ctx, CSD_ERR_SHAPE, "draft T = %d and target T = %d differ", sched_q->T, sched_p->T);
  if (head_q->d.C != head_p->d.C) return fail(ctx, CSD_ERR_SHAPE, "draft C = %d and target C = %d differ", head_q->d.C, head_p->d.C);
  const int C = head_p->d.C, T = sched_p->T;
  if ((rc = check_verify_dims(ctx, B, gamma, C))) return rc;
  if (cap < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "cap = %d must be >= 1", cap);
  if (!u || !xi || !v || !x0 || !mu1_q || !mu1_p || !logratio || !n_accept || !x_new || !n_prop || !flags || !cap_hits)
    return fail(ctx, CSD_ERR_INVALID_ARG, "null array argument");
  if (bonus && (!z_next || !x_T_next || !eps_next || !x_bonus)) return fail(ctx, CSD_ERR_INVALID_ARG, "z_next / x_T_next / eps_next / x_bonus is null");
  CSD_DEVICE(ctx);
  const int Rp = bonus ? R + B : R;    // token rows of the target chain
  // workspaces first (growing one synchronises), then fork the two chains
  if ((rc = ensure_ws(ctx, ctx->ws[0], head_q->d, R * (cfg ? 2 : 1), R, sched_q->T))) return rc;
  if ((rc = ensure_ws(ctx, ctx->ws[1], head_p->d, Rp * (cfg ? 2 : 1), Rp, sched_p->T))) return rc;
  if (bonus && (rc = ensure_side(ctx, ctx->bn, bonus_buf_bytes(head_p->d, Rp, cfg, T), "the bonus rows"))) return rc;
  // Few rows in small-batch mode: each chain is one persistent kernel that wants the whole GPU, so the two run one
  // after the other on the context's stream (the same kernels, hence the same bits, as the separate calls).
  const bool seq = ctx->chain_mode == CSD_CHAIN_SMALL_BATCH && Rp * (cfg ? 2 : 1) <= kSbRows && head_q->sb_ready && head_p->sb_ready;
  if (!seq) {
    CSD_CUDA(ctx, cudaEventRecord(ctx->ev_fork, ctx->stream));
    for (int i = 0; i < 2; ++i) CSD_CUDA(ctx, cudaStreamWaitEvent(ctx->side[i], ctx->ev_fork, 0));
  }
  // the two chains' launches are interleaved step by step so that neither stream starves
  // the chain with more work per row goes to the higher-priority stream
  const double wq = static_cast<double>(head_q->d.L) * head_q->d.W * head_q->d.W, wp = static_cast<double>(head_p->d.L) * head_p->d.W * head_p->d.W;
  const int sq = wq > wp ? 1 : 0;
  cudaStream_t st_q = seq ? ctx->stream : ctx->side[sq], st_p = seq ? ctx->stream : ctx->side[1 - sq];
  BonusBuf bb{};
  if (bonus && (rc = gather_bonus_inputs(ctx, st_p, head_p->d, R, B, cfg, T, z_p, x_T, eps, z_next, x_T_next, eps_next, bb))) return rc;
  Chain cq{ctx, 0, st_q, head_q, sched_q, R, cfg, cfg_scale, z_q, x_T, eps, 1, x0, mu1_q, nullptr};
  Chain cp = bonus ? Chain{ctx, 1, st_p, head_p, sched_p, Rp, cfg, cfg_scale, bb.z, bb.x_T, bb.eps, 1, bb.x0, bb.mu1, nullptr}
                   : Chain{ctx, 1, st_p, head_p, sched_p, R, cfg, cfg_scale, z_p, x_T, eps, 0, nullptr, mu1_p, nullptr};
  cq.chains = cp.chains = seq ? 1 : 2;
  rc = cp.begin();
  int rc2 = cq.begin();
  for (int t = sched_p->T; t >= 1 && !rc && !rc2; --t) {
    rc = cp.step(t);
    if (!rc) rc2 = cq.step(t);
  }
  if (bonus && !rc) CSD_CUDA(ctx, cudaMemcpyAsync(mu1_p, bb.mu1, static_cast<size_t>(R) * C * 4, cudaMemcpyDeviceToDevice, st_p));
  for (int i = 0; i < 2 && !seq; ++i) {
    CSD_CUDA(ctx, cudaEventRecord(ctx->ev_done[i], ctx->side[i]));
    CSD_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, ctx->ev_done[i], 0));
  }
  if (rc) return rc;
  if (rc2) return rc2;
  const double ls = log_sigma_term(sched_q, sched_p, C);
  rc = accept_scan(ctx, ctx->stream, B, gamma, C, ls, sched_p->sigma[0], sched_q->sigma[0], x0, mu1_q, mu1_p, u, logratio,
                   n_accept, accept_mask);
  if (rc) return rc;
  if (bonus) {
    bonus_select_kernel<<<(B * C + 255) / 256, 256, 0, ctx->stream>>>(B, C, gamma, n_accept, bb.x0 + static_cast<size_t>(R) * C, x_bonus, taken);
    ctx->launches++;
    CSD_CUDA(ctx, cudaGetLastError());
  }
  return resample(ctx, ctx->stream, B, gamma, C, cap, ls, sched_p->sigma[0], sched_q->sigma[0], n_accept, mu1_p, mu1_q, xi,
                  v, x_new, n_prop, flags, cap_hits);
}

int csd_round(csd_ctx* ctx, const csd_head* head_q, const csd_head* head_p, const csd_schedule* sched_q,
              const csd_schedule* sched_p, int B, int gamma, int cfg, float cfg_scale, int cap, const float* z_q,
              const float* z_p, const float* x_T, const float* eps, const float* u, const float* xi, const float* v,
              float* x0, float* mu1_q, float* mu1_p, float* logratio, int32_t* n_accept, uint32_t* accept_mask,
              float* x_new, int32_t* n_prop, uint32_t* flags, int32_t* cap_hits) {
  return round_impl(ctx, head_q, head_p, sched_q, sched_p, B, gamma, cfg, cfg_scale, cap, z_q, z_p, x_T, eps, u, xi, v, x0,
                    mu1_q, mu1_p, logratio, n_accept, accept_mask, x_new, n_prop, flags, cap_hits, false, nullptr, nullptr,
                    nullptr, nullptr, nullptr);
}

int csd_round_bonus(csd_ctx* ctx, const csd_head* head_q, const csd_head* head_p, const csd_schedule* sched_q,
                    const csd_schedule* sched_p, int B, int gamma, int cfg, float cfg_scale, int cap, const float* z_q,
                    const float* z_p, const float* x_T, const float* eps, const float* u, const float* xi, const float* v,
                    const float* z_next, const float* x_T_next, const float* eps_next, float* x0, float* mu1_q,
                    float* mu1_p, float* logratio, int32_t* n_accept, uint32_t* accept_mask, float* x_new,
                    int32_t* n_prop, uint32_t* flags, int32_t* cap_hits, float* x_bonus, uint32_t* taken) {
  return round_impl(ctx, head_q, head_p, sched_q, sched_p, B, gamma, cfg, cfg_scale, cap, z_q, z_p, x_T, eps, u, xi, v, x0,
                    mu1_q, mu1_p, logratio, n_accept, accept_mask, x_new, n_prop, flags, cap_hits, true, z_next, x_T_next,
                    eps_next, x_bonus, taken);
}

// ------------------------------------------------------------------ heads that predict their variances
int csd_schedule_lv_ddpm(int T, const double* beta, double tau, float* a, float* b, float* lv_min, float* lv_max) {
  if (T < 1 || !beta || !a || !b || !lv_min || !lv_max || !(tau > 0.0)) return CSD_ERR_INVALID_ARG;
  double abar = 1.0, abar_prev = 1.0;
  for (int t = 0; t < T; ++t) {
    if (!(beta[t] > 0.0 && beta[t] < 1.0)) return CSD_ERR_INVALID_ARG;
    const double alpha = 1.0 - beta[t];
    abar_prev = abar;
    abar *= alpha;
    a[t] = static_cast<float>(1.0 / std::sqrt(alpha));
    b[t] = static_cast<float>(beta[t] / (std::sqrt(alpha) * std::sqrt(1.0 - abar)));
    lv_max[t] = static_cast<float>(std::log(beta[t]) + 2.0 * std::log(tau));
    // posterior variance beta_t (1 - abar_{t-1}) / (1 - abar_t); zero at t = 1, which borrows the value of t = 2 below
    if (t > 0) lv_min[t] = static_cast<float>(std::log(beta[t] * (1.0 - abar_prev) / (1.0 - abar)) + 2.0 * std::log(tau));
  }
  lv_min[0] = T > 1 ? lv_min[1] : lv_max[0];
  return CSD_OK;
}

int csd_draft_denoise_lv(csd_ctx* ctx, const csd_head* head, const csd_schedule_lv* sched, int R, int cfg,
                         float cfg_scale, const float* z, const float* x_T, const float* eps, float* x0, float* mu1,
                         float* lv1, float* half_logdet, float* x1) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  int rc = check_lv_args(ctx, head, sched, R, cfg, z, x_T, eps);
  if (rc) return rc;
  if (!x0 || !mu1 || !lv1 || !half_logdet) return fail(ctx, CSD_ERR_INVALID_ARG, "x0 / mu1 / lv1 / half_logdet is null");
  CSD_DEVICE(ctx);
  csd_schedule view{sched->T, sched->a, sched->b, nullptr, sched->tfeat};
  Chain c = make_lv_chain(ctx, 0, ctx->stream, head, &view, sched, R, cfg, cfg_scale, z, x_T, eps, 1, x0, mu1, lv1,
                          half_logdet, x1);
  rc = c.begin();
  for (int t = sched->T; t >= 1 && !rc; --t) rc = c.step(t);
  return rc;
}

int csd_verify_lv(csd_ctx* ctx, const csd_head* head_p, const csd_schedule_lv* sched_p, int B, int gamma, int cfg,
                  float cfg_scale, const float* z_p, const float* x_T, const float* eps, const float* x0_q,
                  const float* mu1_q, const float* lv1_q, const float* half_logdet_q, const float* u, float* logratio,
                  int32_t* n_accept, uint32_t* accept_mask, float* mu1_p, float* lv1_p, float* half_logdet_p,
                  float* log_sigma_rows) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  if (B < 1 || gamma < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "B = %d and gamma = %d must be >= 1", B, gamma);
  int rc = check_lv_args(ctx, head_p, sched_p, B * gamma, cfg, z_p, x_T, eps);
  if (rc) return rc;
  if ((rc = check_verify_dims(ctx, B, gamma, head_p->d.C))) return rc;
  if (!x0_q || !mu1_q || !lv1_q || !half_logdet_q || !u || !logratio || !n_accept || !mu1_p || !lv1_p || !half_logdet_p ||
      !log_sigma_rows)
    return fail(ctx, CSD_ERR_INVALID_ARG, "null array argument");
  CSD_DEVICE(ctx);
  csd_schedule view{sched_p->T, sched_p->a, sched_p->b, nullptr, sched_p->tfeat};
  Chain c = make_lv_chain(ctx, 1, ctx->stream, head_p, &view, sched_p, B * gamma, cfg, cfg_scale, z_p, x_T, eps, 0,
                          nullptr, mu1_p, lv1_p, half_logdet_p, nullptr);
  rc = c.begin();
  for (int t = sched_p->T; t >= 1 && !rc; --t) rc = c.step(t);
  if (rc) return rc;
  return accept_scan_lv(ctx, ctx->stream, B, gamma, head_p->d.C, x0_q, mu1_q, lv1_q, half_logdet_q, mu1_p, lv1_p,
                        half_logdet_p, u, logratio, log_sigma_rows, n_accept, accept_mask);
}

int csd_resample_lv(csd_ctx* ctx, int B, int gamma, int C, int cap, const float* log_sigma_rows, const int32_t* n_accept,
                    const float* mu1_p, const float* lv1_p, const float* mu1_q, const float* lv1_q, const float* xi,
                    const float* v, float* x_new, int32_t* n_prop, uint32_t* flags, int32_t* cap_hits) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  int rc = check_verify_dims(ctx, B, gamma, C);
  if (rc) return rc;
  if (cap < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "cap = %d must be >= 1", cap);
  if (!log_sigma_rows || !n_accept || !mu1_p || !lv1_p || !mu1_q || !lv1_q || !xi || !v || !x_new || !n_prop || !flags || !cap_hits)
    return fail(ctx, CSD_ERR_INVALID_ARG, "null array argument");
  CSD_DEVICE(ctx);
  return resample_lv(ctx, ctx->stream, B, gamma, C, cap, log_sigma_rows, n_accept, mu1_p, lv1_p, mu1_q, lv1_q, xi, v, x_new,
                     n_prop, flags, cap_hits);
}

int csd_round_lv(csd_ctx* ctx, const csd_head* head_q, const csd_head* head_p, const csd_schedule_lv* sched_q,
                 const csd_schedule_lv* sched_p, int B, int gamma, int cfg, float cfg_scale, int cap, const float* z_q,
                 const float* z_p, const float* x_T, const float* eps, const float* u, const float* xi, const float* v,
                 float* x0, float* mu1_q, float* lv1_q, float* half_logdet_q, float* mu1_p, float* lv1_p,
                 float* half_logdet_p, float* log_sigma_rows, float* logratio, int32_t* n_accept, uint32_t* accept_mask,
                 float* x_new, int32_t* n_prop, uint32_t* flags, int32_t* cap_hits) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  if (B < 1 || gamma < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "B = %d and gamma = %d must be >= 1", B, gamma);
  const int R = B * gamma;
  int rc = check_lv_args(ctx, head_q, sched_q, R, cfg, z_q, x_T, eps);
  if (rc) return rc;
  if ((rc = check_lv_args(ctx, head_p, sched_p, R, cfg, z_p, x_T, eps))) return rc;
  if (sched_q->T != sched_p->T) return fail(ctx, CSD_ERR_SHAPE, "draft T = %d and target T = %d differ", sched_q->T, sched_p->T);
  if (head_q->d.C != head_p->d.C) return fail(ctx, CSD_ERR_SHAPE, "draft C = %d and target C = %d differ", head_q->d.C, head_p->d.C);
  const int C = head_p->d.C;
  if ((rc = check_verify_dims(ctx, B, gamma, C))) return rc;
  if (cap < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "cap = %d must be >= 1", cap);
  if (!u || !xi || !v || !x0 || !mu1_q || !lv1_q || !half_logdet_q || !mu1_p || !lv1_p || !half_logdet_p || !log_sigma_rows ||
      !logratio || !n_accept || !x_new || !n_prop || !flags || !cap_hits)
    return fail(ctx, CSD_ERR_INVALID_ARG, "null array argument");
  CSD_DEVICE(ctx);
  if ((rc = ensure_ws(ctx, ctx->ws[0], head_q->d, R * (cfg ? 2 : 1), R, sched_q->T))) return rc;
  if ((rc = ensure_ws(ctx, ctx->ws[1], head_p->d, R * (cfg ? 2 : 1), R, sched_p->T))) return rc;
  CSD_CUDA(ctx, cudaEventRecord(ctx->ev_fork, ctx->stream));
  for (int i = 0; i < 2; ++i) CSD_CUDA(ctx, cudaStreamWaitEvent(ctx->side[i], ctx->ev_fork, 0));
  const double wq = static_cast<double>(head_q->d.L) * head_q->d.W * head_q->d.W, wp = static_cast<double>(head_p->d.L) * head_p->d.W * head_p->d.W;
  const int sq = wq > wp ? 1 : 0;
  csd_schedule vq{sched_q->T, sched_q->a, sched_q->b, nullptr, sched_q->tfeat}, vp{sched_p->T, sched_p->a, sched_p->b, nullptr, sched_p->tfeat};
  Chain cq = make_lv_chain(ctx, 0, ctx->side[sq], head_q, &vq, sched_q, R, cfg, cfg_scale, z_q, x_T, eps, 1, x0, mu1_q, lv1_q,
                           half_logdet_q, nullptr);
  Chain cp = make_lv_chain(ctx, 1, ctx->side[1 - sq], head_p, &vp, sched_p, R, cfg, cfg_scale, z_p, x_T, eps, 0, nullptr, mu1_p,
                           lv1_p, half_logdet_p, nullptr);
  cq.chains = cp.chains = 2;
  rc = cp.begin();
  int rc2 = cq.begin();
  for (int t = sched_p->T; t >= 1 && !rc && !rc2; --t) {
    rc = cp.step(t);
    if (!rc) rc2 = cq.step(t);
  }
  for (int i = 0; i < 2; ++i) {
    CSD_CUDA(ctx, cudaEventRecord(ctx->ev_done[i], ctx->side[i]));
    CSD_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, ctx->ev_done[i], 0));
  }
  if (rc) return rc;
  if (rc2) return rc2;
  rc = accept_scan_lv(ctx, ctx->stream, B, gamma, C, x0, mu1_q, lv1_q, half_logdet_q, mu1_p, lv1_p, half_logdet_p, u, logratio,
                      log_sigma_rows, n_accept, accept_mask);
  if (rc) return rc;
  return resample_lv(ctx, ctx->stream, B, gamma, C, cap, log_sigma_rows, n_accept, mu1_p, lv1_p, mu1_q, lv1_q, xi, v, x_new,
                     n_prop, flags, cap_hits);
}

// ------------------------------------------------------------------ explicit Gaussian-mixture heads
static int check_gmm(csd_ctx* ctx, const csd_gmm* m, const char* what) {
  if (!m || !m->logw || !m->mu || !m->log_sigma) return fail(ctx, CSD_ERR_INVALID_ARG, "%s mixture or one of its arrays is null", what);
  if (m->K < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "%s mixture has K = %d components", what, m->K);
  return CSD_OK;
}
static GmmView gmm_view(const csd_gmm* m) { return GmmView{m->K, m->logw, m->mu, m->log_sigma}; }

int csd_gmm_draft_sample(csd_ctx* ctx, int R, int C, const csd_gmm* q, const float* u_comp, const float* noise, float* x,
                         int32_t* comp) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  int rc = check_gmm(ctx, q, "draft");
  if (rc) return rc;
  if (R < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "row count %d must be >= 1", R);
  if (C < 1 || C > 32) return fail(ctx, CSD_ERR_UNSUPPORTED, "token dim C = %d must be in [1, 32]", C);
  if (!u_comp || !noise || !x) return fail(ctx, CSD_ERR_INVALID_ARG, "null array argument");
  CSD_DEVICE(ctx);
  gmm_sample_kernel<<<(R + 3) / 4, 128, 0, ctx->stream>>>(R, C, gmm_view(q), u_comp, noise, x, comp);
  ctx->launches++;
  CSD_CUDA(ctx, cudaGetLastError());
  return CSD_OK;
}

int csd_gmm_verify(csd_ctx* ctx, int B, int gamma, int C, const csd_gmm* q, const csd_gmm* p, const float* x,
                   const float* u, float* logratio, int32_t* n_accept, uint32_t* accept_mask) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  int rc = check_gmm(ctx, q, "draft");
  if (rc || (rc = check_gmm(ctx, p, "target"))) return rc;
  if (B < 1 || gamma < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "B = %d and gamma = %d must be >= 1", B, gamma);
  if (gamma > 32) return fail(ctx, CSD_ERR_UNSUPPORTED, "gamma = %d exceeds 32", gamma);
  if (C < 1 || C > 32) return fail(ctx, CSD_ERR_UNSUPPORTED, "token dim C = %d must be in [1, 32]", C);
  if (!x || !u || !logratio || !n_accept) return fail(ctx, CSD_ERR_INVALID_ARG, "null array argument");
  CSD_DEVICE(ctx);
  gmm_verify_kernel<<<B, 32 * gamma, 0, ctx->stream>>>(B, gamma, C, gmm_view(q), gmm_view(p), x, u, logratio, n_accept, accept_mask);
  ctx->launches++;
  CSD_CUDA(ctx, cudaGetLastError());
  return CSD_OK;
}

int csd_gmm_resample(csd_ctx* ctx, int B, int gamma, int C, int cap, const csd_gmm* q, const csd_gmm* p,
                     const int32_t* n_accept, const float* w, const float* xi, const float* v, float* x_new,
                     int32_t* n_prop, uint32_t* flags, int32_t* cap_hits) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  int rc = check_gmm(ctx, q, "draft");
  if (rc || (rc = check_gmm(ctx, p, "target"))) return rc;
  if (B < 1 || gamma < 1 || gamma > 32) return fail(ctx, B < 1 || gamma < 1 ? CSD_ERR_INVALID_ARG : CSD_ERR_UNSUPPORTED, "B = %d, gamma = %d: need B >= 1 and 1 <= gamma <= 32", B, gamma);
  if (C < 1 || C > 32) return fail(ctx, CSD_ERR_UNSUPPORTED, "token dim C = %d must be in [1, 32]", C);
  if (cap < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "cap = %d must be >= 1", cap);
  if (!n_accept || !w || !xi || !v || !x_new || !n_prop || !flags || !cap_hits) return fail(ctx, CSD_ERR_INVALID_ARG, "null array argument");
  CSD_DEVICE(ctx);
  CSD_CUDA(ctx, cudaMemsetAsync(cap_hits, 0, sizeof(int32_t), ctx->stream));
  gmm_resample_kernel<<<(B + 3) / 4, 128, 0, ctx->stream>>>(B, gamma, C, cap, gmm_view(q), gmm_view(p), n_accept, w, xi, v, x_new,
                                                            n_prop, flags, cap_hits);
  ctx->launches++;
  CSD_CUDA(ctx, cudaGetLastError());
  return CSD_OK;
}

int csd_round_host(csd_ctx* ctx, const csd_head* head_q, const csd_head* head_p, const csd_schedule* sched_q,
                   const csd_schedule* sched_p, int B, int gamma, int cfg, float cfg_scale, int cap, const float* z_q,
                   const float* z_p, const float* x_T, const float* eps, const float* u, const float* xi,
                   const float* v, float* x0, float* mu1_q, float* mu1_p, float* logratio, int32_t* n_accept,
                   uint32_t* accept_mask, float* x_new, int32_t* n_prop, uint32_t* flags, int32_t* cap_hits) {
  if (!ctx) return CSD_ERR_INVALID_ARG;
  if (!head_q || !head_p || !sched_q || !sched_p) return fail(ctx, CSD_ERR_INVALID_ARG, "head / schedule is null");
  if (B < 1 || gamma < 1 || cap < 1) return fail(ctx, CSD_ERR_INVALID_ARG, "B, gamma, cap must be >= 1");
  if (!z_q || !z_p || !x_T || !eps || !u || !xi || !v || !x0 || !mu1_q || !mu1_p || !logratio || !n_accept || !x_new ||
      !n_prop || !flags || !cap_hits)
    return fail(ctx, CSD_ERR_INVALID_ARG, "null array argument");
  if (sched_q->T < 1 || sched_q->T != sched_p->T) return fail(ctx, CSD_ERR_SHAPE, "schedules disagree on T");
  CSD_DEVICE(ctx);
  const size_t R = static_cast<size_t>(B) * gamma, Rh = R * (cfg ? 2 : 1), C = head_p->d.C, T = sched_p->T;
  struct Item { const void* src; void* dst; size_t bytes; size_t off; bool in; };
  Item items[] = {
      {z_q, nullptr, Rh * head_q->d.Dz * 4, 0, true}, {z_p, nullptr, Rh * head_p->d.Dz * 4, 0, true},
      {x_T, nullptr, R * C * 4, 0, true},             {eps, nullptr, T * R * C * 4, 0, true},
      {u, nullptr, R * 4, 0, true},                   {xi, nullptr, static_cast<size_t>(B) * cap * C * 4, 0, true},
      {v, nullptr, static_cast<size_t>(B) * cap * 4, 0, true},
      {nullptr, x0, R * C * 4, 0, false},             {nullptr, mu1_q, R * C * 4, 0, false},
      {nullptr, mu1_p, R * C * 4, 0, false},          {nullptr, logratio, R * 4, 0, false},
      {nullptr, n_accept, static_cast<size_t>(B) * 4, 0, false},
      {nullptr, accept_mask, static_cast<size_t>(B) * 4, 0, false},
      {nullptr, x_new, static_cast<size_t>(B) * C * 4, 0, false},
      {nullptr, n_prop, static_cast<size_t>(B) * 4, 0, false}, {nullptr, flags, static_cast<size_t>(B) * 4, 0, false},
      {nullptr, cap_hits, 4, 0, false}};
  size_t total = 0;
  for (Item& it : items) { it.off = total; total = align_up(total + it.bytes, 256); }
  if (total > ctx->io.cap) {
    CSD_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (ctx->io.base) CSD_CUDA(ctx, cudaFree(ctx->io.base));
    ctx->io.base = nullptr; ctx->io.cap = 0;
    if (cudaMalloc(&ctx->io.base, total) != cudaSuccess) { cudaGetLastError(); return fail(ctx, CSD_ERR_WORKSPACE, "cannot allocate %zu bytes for the host-call mirrors", total); }
    ctx->io.cap = total;
  }
  char* base = static_cast<char*>(ctx->io.base);
  auto dp = [&](int i) { return base + items[i].off; };
  for (int i = 0; i < 7; ++i) CSD_CUDA(ctx, cudaMemcpyAsync(dp(i), items[i].src, items[i].bytes, cudaMemcpyHostToDevice, ctx->stream));
  CSD_CUDA(ctx, cudaMemsetAsync(dp(13), 0, items[13].bytes, ctx->stream));  // x_new: rows that are not resampled read 0
  int rc = csd_round(ctx, head_q, head_p, sched_q, sched_p, B, gamma, cfg, cfg_scale, cap, (const float*)dp(0),
                     (const float*)dp(1), (const float*)dp(2), (const float*)dp(3), (const float*)dp(4),
                     (const float*)dp(5), (const float*)dp(6), (float*)dp(7), (float*)dp(8), (float*)dp(9), (float*)dp(10),
                     (int32_t*)dp(11), (uint32_t*)dp(12), (float*)dp(13), (int32_t*)dp(14), (uint32_t*)dp(15),
                     (int32_t*)dp(16));
  if (rc) return rc;
  for (int i = 7; i < 17; ++i)
    if (items[i].dst) CSD_CUDA(ctx, cudaMemcpyAsync(items[i].dst, dp(i), items[i].bytes, cudaMemcpyDeviceToHost, ctx->stream));
  return csd_sync(ctx);
}

}  // extern "C"
