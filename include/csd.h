/*
 * csd.h - C ABI of the continuous speculative decoding (CSD) hot path for NVIDIA B200 (sm_100a).
 *
 * The library evaluates, for a batch of independent token rows, what one round of Algorithm 1
 * ("ContinuousSpeculativeDecodingStep") of "Continuous Speculative Decoding for Autoregressive
 * Image Generation" needs from the per-token diffusion heads, with the AR transformer backbones
 * left to the caller: their output vectors z, the Gaussian noise, the uniforms, the noise schedule
 * and the head weights are all inputs.
 *
 * Conventions
 *   B sequences, gamma draft tokens per sequence, R = B*gamma token rows, row r = b*gamma + i.
 *   cfg = 1 doubles the head rows for classifier-free guidance (Appendix "Classifier-Free
 *   Guidance"): z has 2R rows, [conditional rows | unconditional rows]; both halves see the
 *   same x_t and eps_hat = eps_u + cfg_scale * (eps_c - eps_u).
 *   C token dim, W head width, L residual blocks, Dz condition dim, F timestep-feature dim, T steps.
 *   Every array is dense row-major.  "device" = pointer to GPU global memory of the context's
 *   device, "host" = ordinary host memory.  The library never frees or keeps caller memory
 *   beyond the call (host arrays are copied before the call returns; device arrays are read by
 *   the kernels the call enqueues and must stay valid until those have run).
 *   All work is enqueued on the stream given to csd_create(); calls return without
 *   synchronising unless stated.  Device-side error flags (for instance a bounded wait that ran
 *   out) are reported by csd_sync().
 *
 * Head evaluated per head row and step t (eps-prediction network of Eq. 3; the layout below is
 * this library's specification, the paper does not describe the head's inside):
 *   cz = Wz z + bz ;  te_t = Wt2 SiLU(Wt1 tfeat_t + bt1) + bt2 ;  s = SiLU(cz + te_t)
 *   h = Win x_t + bin
 *   for k < L: (shift|scale|gate) = Wada_k s + bada_k ; u = LN(h)(1+scale)+shift ;
 *              h = h + gate * (W2_k SiLU(W1_k u + b1_k) + b2_k)
 *   (shift|scale) = Wfada s + bfada ;  eps_hat = Wout (LN(h)(1+scale)+shift) + bout
 *   LN: no affine, eps 1e-6, biased variance over W.
 *
 * Errors: every function returns CSD_OK (0) or a negative code; nothing aborts, throws or traps.
 * csd_last_error() returns a description of the most recent failure on that context.
 */
#ifndef CSD_H_
#define CSD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct csd_ctx csd_ctx;
typedef struct csd_head csd_head;

enum {
  CSD_OK = 0,
  CSD_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, bad enum                         */
  CSD_ERR_SHAPE = -2,       /* dims of heads / schedules / calls do not agree                    */
  CSD_ERR_UNSUPPORTED = -3, /* e.g. W not a multiple of 128, gamma > 32, C > 16, not an sm_100 GPU */
  CSD_ERR_WORKSPACE = -4,   /* device memory for the workspace or weights could not be had      */
  CSD_ERR_CUDA = -5,        /* a CUDA runtime/driver call failed                                 */
  CSD_ERR_TIMEOUT = -6,     /* a bounded device-side wait gave up (reported by csd_sync)         */
  CSD_ERR_NONFINITE = -7    /* a state or mean of a denoising step was inf or NaN (reported by csd_sync) */
};

enum { CSD_F32 = 0, CSD_BF16 = 1, CSD_F16 = 2 };

/* Shape and arithmetic of one head.
 * CSD_F32 : fp32 weights and activations on plain FMA units.
 * CSD_BF16: tcgen05 tensor cores, both GEMM operands bf16 (weights and activations rounded to
 *           bf16), fp32 accumulation in TMEM.
 * CSD_F16 : the same kernels with both operands IEEE fp16.  Meant for weights whose VALUES are
 *           bf16-representable: such a value is exact in fp16 when |w| >= 2^-17 (else it is off
 *           by at most 2^-25), and activations keep 11 significant bits instead of 8, which the
 *           long, error-amplifying T-step trajectories need (a tensor-core instruction takes
 *           both operands in one 16-bit format).  Activations must stay below 65504 in magnitude: a
 *           larger one is rounded to infinity, reaches the step update as inf or NaN and is reported by
 *           csd_sync as CSD_ERR_NONFINITE (nothing faults; the outputs of that call are not usable).
 *           Heads whose activations can grow that large (weights far above Xavier scale) take CSD_BF16
 *           (fp32 range, 8 significant bits) or CSD_F32.
 * In all three the residual stream, LayerNorm statistics, x_t, mu and the densities are fp32. */
typedef struct {
  int C, W, L, Dz, F;
  int dtype;   /* CSD_F32 | CSD_BF16 | CSD_F16 */
  int var_out; /* 0: the head predicts eps_hat (C outputs) and the transition's variance is the schedule's fixed
                  sigma_t^2; 1: the head also predicts the diagonal of Sigma_theta(x_t, t) of Eq. 3 (2C outputs,
                  Wout [2C, W], bout [2C]: rows C..2C are the variance parameter w) - such a head is used with the
                  _lv calls below */
} csd_head_desc;

/* HOST pointers to fp32 parameters, each matrix row-major [out, in]:
 * Wz[W,Dz] bz[W] Wt1[W,F] bt1[W] Wt2[W,W] bt2[W] Win[W,C] bin[W] Wada[L,3W,W] bada[L,3W]
 * W1[L,W,W] b1[L,W] W2[L,W,W] b2[L,W] Wfada[2W,W] bfada[2W] Wout[C,W] bout[C]  (Wout[2C,W] bout[2C] if var_out).
 * For CSD_BF16 / CSD_F16 heads the matrices are converted to that format (round to nearest
 * even); callers that want bit-defined results pass values that are already representable. */
typedef struct {
  const float *Wz, *bz, *Wt1, *bt1, *Wt2, *bt2, *Win, *bin;
  const float *Wada, *bada, *W1, *b1, *W2, *b2, *Wfada, *bfada, *Wout, *bout;
} csd_head_weights;

/* Reverse-process coefficients of a T-step sampler whose transition is the Gaussian of Eq. 3
 * with isotropic variance: mu_t = a[t-1] x_t - b[t-1] eps_hat, x_{t-1} = mu_t + sigma[t-1] eps_t.
 * sigma already includes the sampling temperature (Appendix "Temperature").
 * a, b, sigma: HOST arrays [T].  tfeat: DEVICE array [T, F], row t-1 = features of timestep t. */
typedef struct {
  int T;
  const float *a, *b, *sigma;
  const float *tfeat;
} csd_schedule;

/* Context: owns a growable device workspace and the stream association.  `cuda_stream` is a
 * cudaStream_t (NULL = legacy default stream).  csd_destroy synchronises the stream and frees.
 * Several contexts, also on different devices (ordinals below 64), may live in one process.  Every call
 * makes the context's device current while it runs and puts the caller's current device back on return. */
int csd_create(csd_ctx **out, int device, void *cuda_stream);
int csd_destroy(csd_ctx *ctx);
const char *csd_last_error(const csd_ctx *ctx);
/* Waits for the context's stream and returns CSD_ERR_TIMEOUT (a bounded wait of some kernel gave up; the
 * message names the waiting role, the wait's site in the kernel, its iteration and the thread block),
 * CSD_ERR_NONFINITE (see csd_head_desc) or CSD_ERR_CUDA if a kernel of an earlier call raised its status
 * word, else CSD_OK.  Clears the status.  After a failed wait every later launch of the context returns
 * at once until csd_sync has been called. */
int csd_sync(csd_ctx *ctx);
/* Every device-side wait of the library (on an mbarrier of a TMA / MMA / epilogue pipeline) is bounded:
 * after `cycles` SM clock cycles (default 4e9, about two seconds; cycles <= 0 restores the default) it
 * gives up and raises the status csd_sync reports.  The limit is one value per GPU and process (all
 * contexts on that device share it).  Synchronises the context's streams. */
int csd_set_wait_limit(csd_ctx *ctx, int64_t cycles);
/* Diagnostic: enqueues one tiny kernel whose only thread waits on a barrier nobody arrives at, i.e. a wait
 * that is certain to run into the limit above.  Used to check the reporting path (csd_sync returns
 * CSD_ERR_TIMEOUT, "wait self-test") without disturbing the GPU: nothing faults or traps, and the wait
 * ends at the limit.  Set a short limit first (1e5 cycles) or the call takes the default two seconds. */
int csd_selftest_wait_timeout(csd_ctx *ctx);
/* Number of kernels this context has launched so far (bookkeeping for benchmarks). */
int64_t csd_launch_count(const csd_ctx *ctx);

/* How the blocks of a denoising chain (the T steps of Eq. 3 for one head) are split into kernels.
 *   CSD_CHAIN_LAYERS  (default): the library picks by size.
 *                     - Layers of one wave of 128 x 128 tiles on a 16-bit head with W = 1024, var_out = 0 and an
 *                       even number of row blocks (128 head rows each: 64 tokens with guidance, 128 without; a few
 *                       hundred to about a thousand head rows) run as ONE persistent kernel per chain: a pair of
 *                       CTAs owns its output tiles for every layer and step, the residual stream stays in tensor
 *                       memory, the CTAs that share rows meet at a counter once per layer.  Draft and target chain
 *                       of csd_round then run side by side without competing for SMs.  Its buffers grow with T
 *                       (the condition vectors of all steps: T x rows x W 16-bit values).  A chain that has the GPU
 *                       to itself (csd_draft_denoise or csd_verify called alone) is about a tenth faster with
 *                       CSD_CHAIN_LAYER_KERNELS, whose kernels spread over the idle SMs; the default is chosen
 *                       per chain, not per call, so that csd_round and the three separate calls give the same bits.
 *                     - Otherwise one kernel per layer, chained with programmatic dependent launch; a layer's
 *                       independent part overlaps its predecessor on otherwise idle SMs.  For 16-bit heads on
 *                       grids of one wave, blocks 2..L run as two kernels instead of three: LayerNorm is folded
 *                       into the first layer's epilogue.
 *                     Folding is algebraically the same function, rounded differently: the layouts agree within
 *                     the parity tolerance, not bit for bit, and which one runs depends on the call's row count.
 *   CSD_CHAIN_LAYER_KERNELS: as CSD_CHAIN_LAYERS without the persistent kernel (layer kernels, folded where
 *                     that applies): what csd_draft_denoise_static always runs.
 *   CSD_CHAIN_LAYERS_PLAIN: layer kernels without the folded blocks (three kernels per block everywhere); a
 *                     row's bits then do not depend on how many rows the call has.
 *   CSD_CHAIN_SMALL_BATCH: as CSD_CHAIN_LAYERS, except that a chain of at most 128 head rows (R (1 + cfg) <= 128)
 *                     on a 16-bit head with W in {512, 1024, 1536} and var_out = 0 runs as ONE persistent kernel
 *                     that spreads every layer over the whole GPU (weights as the MMA's M operand, a cluster of 8
 *                     CTAs per group of 16 rows, the products of the condition vector computed a step ahead by the
 *                     remaining SMs).  This is the calling pattern Alg. 1 forces on the draft model (x_i ~ q_i one
 *                     position at a time), where the layer kernels are bound by kernel latency.  Every block is
 *                     folded, so results agree with the other layouts within the parity tolerance.  The kernel
 *                     needs the GPU to itself: csd_round then runs its two chains one after the other, and two
 *                     contexts should not run such chains at the same time (the kernels would wait for each
 *                     other's SMs until the wait limit and report CSD_ERR_TIMEOUT).
 * Takes effect for calls made after it returns. */
enum { CSD_CHAIN_LAYERS = 0, CSD_CHAIN_SMALL_BATCH = 1, CSD_CHAIN_LAYERS_PLAIN = 2, CSD_CHAIN_LAYER_KERNELS = 3 };
int csd_set_chain_mode(csd_ctx *ctx, int mode);

/* Optional per-launch timing for benchmarks.  csd_profile(ctx, 1) synchronises, clears the records
 * and makes every later GEMM-chain launch of this context be bracketed by CUDA events on the
 * stream it runs on (this costs a little time per launch, so throughput is measured with it
 * off); csd_profile(ctx, 0) switches it off.  csd_profile_read synchronises and sums, for one
 * kernel class, the launches recorded since: their count, device time (ms) and algorithmic FLOPs
 * (2*M*N*K per GEMM).  Classes: 0 condition projection, 1 block MLP first layer (+SiLU),
 * 2 AdaLN modulate (shift|scale), 3 block MLP second layer + gate + residual, 4 final modulate +
 * output projection, 5 per-step boundary kernel, 6 small-batch chain kernel. */
int csd_profile(csd_ctx *ctx, int enable);
int csd_profile_read(csd_ctx *ctx, int kernel_class, int64_t *launches, double *total_ms,
                     double *total_flops);

/* Host-only helpers: the schedules of the samplers the paper uses, as the coefficient arrays csd_schedule
 * takes.  No GPU work, no context; all pointers are HOST arrays; return CSD_OK or CSD_ERR_INVALID_ARG.
 *
 * csd_schedule_ddpm: the T-step DDPM reverse process behind Eq. 3 with the eps-prediction mean and fixed
 * isotropic variance: alpha_t = 1 - beta_t, abar_t = prod_{s<=t} alpha_s,
 *   a[t-1] = 1/sqrt(alpha_t),  b[t-1] = beta_t / (sqrt(alpha_t) sqrt(1 - abar_t)),  sigma[t-1] = tau sqrt(beta_t)
 * (tau = sampling temperature, Appendix "Temperature").  beta [T] in (0,1); a, b, sigma [T] out. */
int csd_schedule_ddpm(int T, const double *beta, double tau, float *a, float *b, float *sigma);
/* csd_schedule_ddim: the DDIM sampler of the appendix "More Variants of Diffusion Model" (Table 9 runs 100
 * steps) on the ascending sub-sequence steps[0..n_steps) (1-based timesteps) of a T_full-step DDPM, with
 * stochasticity eta in (0, 1] (eta = 0 has no density to take ratios of).  With prv / cur = abar of the
 * previous / current kept timestep:  sigma = eta sqrt((1-prv)/(1-cur)) sqrt(1 - cur/prv),
 *   a = sqrt(prv/cur),  b = a sqrt(1-cur) - sqrt(1 - prv - sigma^2).
 * Entry k is the (k+1)-th step counted from x_0; the step to x_0 (prv = 1) gets sigma = eta sqrt(1 - cur)
 * around the predicted x_0.  Pass the feature rows of the same timesteps as csd_schedule.tfeat. */
int csd_schedule_ddim(int T_full, const double *beta_full, int n_steps, const int32_t *steps, double eta,
                      float *a, float *b, float *sigma);
/* csd_log_sigma_term: log Sigma of Eq. 7 for fixed isotropic variances,
 * C * sum_{t=2..T} (log sigma_q[t-1] - log sigma_p[t-1]), exactly as csd_verify and csd_round form it. */
int csd_log_sigma_term(int T, const float *sigma_q, const float *sigma_p, int C, double *out);

/* Copies and repacks the weights into device memory owned by the head (synchronous; the caller
 * may free `w` afterwards).  A head belongs to the context it was created with. */
int csd_head_create(csd_ctx *ctx, const csd_head_desc *desc, const csd_head_weights *w, csd_head **out);
int csd_head_destroy(csd_head *head);

/* Draft trajectories (Alg. 1 "x_i ~ q_i"; Eq. 1, Eq. 3; reparameterised sampling of Sec. 3.2):
 * for each of R token rows run t = T..1 of the head given, adding sigma_t eps_t at EVERY step
 * including t = 1, so that x0 = mu1 + sigma_1 eps_1 is a draw from the final-step Gaussian
 * q(x_0 | x_1).  Given the target head this call is also the target-only pre-fill of
 * Sec. 3.2 ("Inconsistency in Autoregressive Process").
 *   z    device [R*(1+cfg), Dz] fp32        x_T  device [R, C]      eps  device [T, R, C]
 *   x0   device [R, C] out                  mu1  device [R, C] out  (mean of the last step)
 *   x1   device [R, C] out or NULL          (state before the last step) */
int csd_draft_denoise(csd_ctx *ctx, const csd_head *head, const csd_schedule *sched, int R, int cfg,
                      float cfg_scale, const float *z, const float *x_T, const float *eps,
                      float *x0, float *mu1, float *x1);

/* csd_draft_denoise without any allocation (the paper has no counterpart: this is a deployment
 * variant of the call above with the same arguments; it runs the layer kernels, so its results are
 * bit-identical to csd_draft_denoise in the modes CSD_CHAIN_LAYER_KERNELS and CSD_CHAIN_LAYERS_PLAIN, and
 * in the default mode whenever that call does not take the persistent chain kernel, whose buffers
 * grow with T and cannot live in a fixed array; otherwise the two agree within the parity tolerance).
 * Who needs it: code that must not, or cannot, reach the CUDA allocator when the call is made -
 * a serving process whose framework has handed all free device memory to its own pool so that
 * cudaMalloc fails, a latency-critical loop where cudaMalloc's implicit device synchronisation is
 * unacceptable, or a sandboxed plug-in that is only allowed to launch kernels.  csd_draft_denoise
 * grows a cudaMalloc'ed workspace on demand; this call instead keeps every intermediate
 * (condition projection, activations, residual stream, LayerNorm partials, eps partial sums, x_t)
 * in one 8 MiB array that is compiled into the library as a static __device__ object, so every
 * GPU that loads the library holds those 8 MiB until the process exits.
 * Limits and rules:
 *   - the call is rejected with CSD_ERR_WORKSPACE, before anything is enqueued, if its
 *     intermediates do not fit in 8 MiB (roughly R*(1+cfg) <= 128 head rows at W = 1536, T = 100;
 *     the error text gives the exact byte count);
 *   - it calls no cudaMalloc / cudaFree and no allocating library routine; profiling
 *     (csd_profile) must be off, since recording creates CUDA events;
 *   - the first call on a device looks up the array's device address (cudaGetSymbolAddress); make
 *     that first call outside any stream capture;
 *   - all calls, from every context of the process on that GPU, share the one array, which keeps
 *     the previous call's contents (nothing in it needs to start at zero: each buffer is written
 *     before it is read).  Two such calls that overlap on the GPU (different streams or contexts)
 *     race on it and give wrong results: serialise them. */
int csd_draft_denoise_static(csd_ctx *ctx, const csd_head *head, const csd_schedule *sched, int R,
                             int cfg, float cfg_scale, const float *z, const float *x_T,
                             const float *eps, float *x0, float *mu1, float *x1);

/* Verification (Alg. 1: target run with the draft's noise, Sigma, ratios, accepted count).
 * Runs the target head on the SAME x_T and eps as the draft call (denoising trajectory
 * alignment, Theorem 1) for t = T..1 without sampling x_0, then per row
 *   logratio = log Sigma + log N(x0; mu1_p, sigma_p,1^2 I) - log N(x0; mu1_q, sigma_q,1^2 I)
 * (Eq. 8) with log Sigma = C * sum_{t=2..T} (log sigma_q,t - log sigma_p,t) (Eq. 7), accepts
 * position i iff log u[b,i] <= logratio[b,i] and returns n_accept[b] = number of leading accepts.
 *   sched_p: full schedule of the target; sched_q: only T and sigma are read.
 *   z_p device [B*gamma*(1+cfg), Dz_p]; x_T, eps, x0_q, mu1_q device as in the draft call;
 *   u device [B, gamma] in (0,1];  logratio device [B, gamma] out;  n_accept device int32 [B] out;
 *   accept_mask device uint32 [B] out or NULL (bit i = position i accepted);
 *   mu1_p device [B*gamma, C] out. */
int csd_verify(csd_ctx *ctx, const csd_head *head_p, const csd_schedule *sched_p,
               const csd_schedule *sched_q, int B, int gamma, int cfg, float cfg_scale,
               const float *z_p, const float *x_T, const float *eps, const float *x0_q,
               const float *mu1_q, const float *u, float *logratio, int32_t *n_accept,
               uint32_t *accept_mask, float *mu1_p);

/* Only the ratio / accept / prefix part of csd_verify, for callers that already hold mu1_p
 * (no head is evaluated).  log_sigma_term = log Sigma of Eq. 7 (host double). */
int csd_accept_scan(csd_ctx *ctx, int B, int gamma, int C, double log_sigma_term, float sigma1_p,
                    float sigma1_q, const float *x0_q, const float *mu1_q, const float *mu1_p,
                    const float *u, float *logratio, int32_t *n_accept, uint32_t *accept_mask);

/* Verification WITHOUT denoising trajectory alignment (the ablation of the paper's alignment study:
 * the target draws its own noise).  As csd_verify, but the target's chain uses eps_p while the
 * draft's used eps_q, so the per-step exponentials of Eq. 4 no longer cancel into Eq. 7/8: with
 * x^m_{t-1} - mu^m_t = sigma_m,t eps^m_t,
 *   logratio = [Eq. 8 evaluated with this target's mu1_p]
 *              + sum_{t=2..T} (|eps^q_t|^2 - |eps^p_t|^2) / 2.
 * With eps_p == eps_q the extra sum is exactly 0 and the call returns csd_verify's bits.
 *   eps_p, eps_q device [T, B*gamma, C]; everything else as in csd_verify. */
int csd_verify_unaligned(csd_ctx *ctx, const csd_head *head_p, const csd_schedule *sched_p,
                         const csd_schedule *sched_q, int B, int gamma, int cfg, float cfg_scale,
                         const float *z_p, const float *x_T, const float *eps_p, const float *eps_q,
                         const float *x0_q, const float *mu1_q, const float *u, float *logratio,
                         int32_t *n_accept, uint32_t *accept_mask, float *mu1_p);

/* Bonus token (Alg. 1, the branch in which all gamma drafts were accepted: "sample x from p_{gamma+1}").
 * Runs the target head's reverse process (t = T..1, noise at every step, as csd_draft_denoise does) for
 * position gamma+1 of every sequence and keeps the sample where n_accept[b] == gamma.  All B rows are
 * evaluated because n_accept lives on the device; the selection costs no host synchronisation.
 *   z_next device [B*(1+cfg), Dz_p] (the target backbone's output at position gamma+1);
 *   x_T_next device [B, C]; eps_next device [T, B, C]; n_accept device int32 [B] (from csd_verify);
 *   x_bonus device [B, C] out, untouched where n_accept[b] < gamma;
 *   taken device uint32 [B] out or NULL: 1 where a bonus token was written. */
int csd_bonus_token(csd_ctx *ctx, const csd_head *head_p, const csd_schedule *sched_p, int B, int gamma,
                    int cfg, float cfg_scale, const float *z_next, const float *x_T_next,
                    const float *eps_next, const int32_t *n_accept, float *x_bonus, uint32_t *taken);

/* csd_verify with the bonus token folded in.  Alg. 1 obtains p_{gamma+1} from the same parallel target pass that
 * yields p_1..p_gamma, so here the B rows of position gamma+1 ride along as rows R..R+B of the verifying chain
 * (one chain of R + B token rows instead of a second, latency-bound chain of B rows): those rows sample x_0 at
 * the last step, and x_bonus[b] is written where n_accept[b] == gamma.  logratio, n_accept, accept_mask, mu1_p as
 * csd_verify; z_next, x_T_next, eps_next, x_bonus, taken as csd_bonus_token.  The inputs are gathered into a
 * side buffer the library keeps ((R + B) rows of z, x_T, eps).  Results equal csd_verify followed by
 * csd_bonus_token bit for bit with CSD_CHAIN_LAYERS_PLAIN, and within the trajectory tolerance in the default
 * layout (whose folded blocks depend on a call's row count). */
int csd_verify_bonus(csd_ctx *ctx, const csd_head *head_p, const csd_schedule *sched_p,
                     const csd_schedule *sched_q, int B, int gamma, int cfg, float cfg_scale,
                     const float *z_p, const float *x_T, const float *eps, const float *x0_q,
                     const float *mu1_q, const float *u, const float *z_next, const float *x_T_next,
                     const float *eps_next, float *logratio, int32_t *n_accept, uint32_t *accept_mask,
                     float *mu1_p, float *x_bonus, uint32_t *taken);

/* ---- Exact single-path criterion (Eq. 2; Table 1 "p(Y_q)/q(Y_q)") ------------------------------
 * Eq. 2 scores the DRAFT's own trajectory Y_q = (x_T, x^q_{T-1}, ..., x^q_0) under both models:
 *   log p(Y_q)/q(Y_q) = sum_{t=1..T} [ log N(x^q_{t-1}; mu^p_t(x^q_t), sigma_p,t^2 I)
 *                                    - log N(x^q_{t-1}; mu^q_t(x^q_t), sigma_q,t^2 I) ].
 * The paper shows this exact ratio accepts almost nothing and replaces it by Eq. 4; it is provided as the
 * diagnostic the approximated criterion of csd_verify is measured against.
 *
 * csd_draft_denoise_traj: csd_draft_denoise that records the whole trajectory.
 *   traj_x  device [T+1, R, C] out: slot j = x_{T-j} (slot 0 = x_T, slot T = x_0)
 *   traj_mu device [T,   R, C] out: slot j = mu_{T-j} (the mean from which slot j+1 of traj_x was drawn)
 *   other arguments as in csd_draft_denoise; x_0 and mu_1 are the last slots. */
int csd_draft_denoise_traj(csd_ctx *ctx, const csd_head *head, const csd_schedule *sched, int R, int cfg,
                           float cfg_scale, const float *z, const float *x_T, const float *eps,
                           float *traj_x, float *traj_mu);

/* csd_verify_single_path: evaluates the target head at every state of the draft's trajectory and
 * returns the log of Eq. 2 per token, then the accept test and prefix count of Alg. 1 on it
 * (accept iff log u <= logratio).  Given the trajectory, the T target evaluations do not depend on
 * one another: they run as ceil(T / steps_per_pass) passes of the layers over steps_per_pass * R
 * token rows each instead of T dependent steps.  Per step the two quadratic forms are rounded
 * separately, so a target that reproduces the draft's means bit for bit gives exactly 0.
 *   sched_p: full schedule of the target; sched_q: only T and sigma are read (same T).
 *   z_p device [B*gamma*(1+cfg), Dz_p]; traj_x, traj_mu_q device, as written by
 *   csd_draft_denoise_traj for R = B*gamma; u device [B, gamma] in (0,1];
 *   steps_per_pass: 0 = chosen by the library (about 32768 head rows per pass).  The steps are
 *   summed in trajectory order whatever the split; with CSD_CHAIN_LAYERS_PLAIN the result does not
 *   depend on it by a bit, in the default mode the block layout follows a pass's row count and
 *   results of different splits agree within the parity tolerance;
 *   logratio device [B, gamma] out; n_accept device int32 [B] out; accept_mask device uint32 [B]
 *   out or NULL; mu_p_traj device [T, R, C] out or NULL: slot j = the target's mean mu^p_{T-j}(x^q_{T-j}),
 *   the counterpart of traj_mu_q (diagnostic; the per-step terms are formed from exactly these values).
 * The library keeps a side buffer of steps_per_pass * R * C floats besides the chain workspace. */
int csd_verify_single_path(csd_ctx *ctx, const csd_head *head_p, const csd_schedule *sched_p,
                           const csd_schedule *sched_q, int B, int gamma, int cfg, float cfg_scale,
                           const float *z_p, const float *traj_x, const float *traj_mu_q,
                           const float *u, int steps_per_pass, float *logratio, int32_t *n_accept,
                           uint32_t *accept_mask, float *mu_p_traj);

/* Resampling from the modified distribution max(0, p - q)/Z (Eq. 5) by acceptance-rejection with
 * the bound M = 1/Z (Eq. 9-11) in the inference-free form of Corollary 1.  For each sequence with
 * n_accept[b] < gamma, row j = b*gamma + n_accept[b]: for k = 0..cap-1
 *   x' = mu1_p[j] + sigma1_p * xi[b,k];
 *   alpha_s = max(0, 1 - q(x'|x_1^q) / (Sigma p(x'|x_1^p)));   accept iff v[b,k] <= alpha_s.
 * The loop of Alg. 1 is unbounded; here it stops after `cap` proposals, returns the last one and
 * sets bit 1 of flags[b].
 *   n_accept device int32 [B]; mu1_p, mu1_q device [B*gamma, C]; xi device [B, cap, C] ~ N(0,1);
 *   v device [B, cap] in (0,1);  x_new device [B, C] out (untouched where n_accept == gamma);
 *   n_prop device int32 [B] out (0 where nothing was resampled);
 *   flags device uint32 [B] out: bit0 resampled, bit1 cap hit;  cap_hits device int32 [1] out. */
int csd_resample(csd_ctx *ctx, int B, int gamma, int C, int cap, double log_sigma_term,
                 float sigma1_p, float sigma1_q, const int32_t *n_accept, const float *mu1_p,
                 const float *mu1_q, const float *xi, const float *v, float *x_new,
                 int32_t *n_prop, uint32_t *flags, int32_t *cap_hits);

/* One whole round of Alg. 1 = csd_draft_denoise + csd_verify + csd_resample with bit-identical
 * results; the two heads' chains run concurrently on internal streams (they are independent
 * until the final-step densities, Eq. 4) and are joined on the context's stream before return
 * of control to that stream.  Argument meaning as in the three calls. */
int csd_round(csd_ctx *ctx, const csd_head *head_q, const csd_head *head_p,
              const csd_schedule *sched_q, const csd_schedule *sched_p, int B, int gamma, int cfg,
              float cfg_scale, int cap, const float *z_q, const float *z_p, const float *x_T,
              const float *eps, const float *u, const float *xi, const float *v, float *x0,
              float *mu1_q, float *mu1_p, float *logratio, int32_t *n_accept,
              uint32_t *accept_mask, float *x_new, int32_t *n_prop, uint32_t *flags,
              int32_t *cap_hits);

/* ---- Heads that predict their variances (the general transition of Eq. 3) -------------------------
 * Eq. 3 writes the transition as N(x_{t-1}; mu_theta(x_t,t), Sigma_theta(x_t,t)) with both moments predicted by
 * the network the paper cites for it.  A head created with var_out = 1 returns, next to eps_hat, a parameter w
 * per coordinate; the transition's diagonal log-variance interpolates between two per-step bounds,
 *   lv_{t,d} = lv_min[t-1] + (w_d + 1)/2 * (lv_max[t-1] - lv_min[t-1]),   x_{t-1} = mu_t + exp(lv_t / 2) * eps_t.
 * With guidance eps_hat is guided and w is the conditional row's.  Sigma of Eq. 7 is then a per-token product:
 * log Sigma[r] = half_logdet_q[r] - half_logdet_p[r], half_logdet = (1/2) sum_{t=2..T} sum_d lv_{t,d} of a chain;
 * Eq. 8 and Corollary 1 use the diagonal final-step Gaussians N(mu1, diag(exp(lv1))).
 * csd_schedule_lv: a, b, lv_min, lv_max HOST arrays [T]; tfeat DEVICE [T, F].
 * csd_schedule_lv_ddpm (host only): a, b as csd_schedule_ddpm; lv_max = log beta_t, lv_min = log of the posterior
 * variance beta_t (1 - abar_{t-1}) / (1 - abar_t) (its value at t = 2 also for t = 1, where it is zero), both
 * plus 2 log tau. */
typedef struct {
  int T;
  const float *a, *b, *lv_min, *lv_max;
  const float *tfeat;
} csd_schedule_lv;
int csd_schedule_lv_ddpm(int T, const double *beta, double tau, float *a, float *b, float *lv_min, float *lv_max);
/* As csd_draft_denoise; also returns lv1 device [R, C] (log-variance of the last step) and half_logdet device [R]. */
int csd_draft_denoise_lv(csd_ctx *ctx, const csd_head *head, const csd_schedule_lv *sched, int R, int cfg,
                         float cfg_scale, const float *z, const float *x_T, const float *eps, float *x0,
                         float *mu1, float *lv1, float *half_logdet, float *x1);
/* As csd_verify (shared x_T and eps: alignment); takes the draft's lv1_q, half_logdet_q and returns the target's
 * mu1_p, lv1_p [R, C], half_logdet_p [R] and the per-token log_sigma_rows device [R] besides logratio, n_accept, mask. */
int csd_verify_lv(csd_ctx *ctx, const csd_head *head_p, const csd_schedule_lv *sched_p, int B, int gamma, int cfg,
                  float cfg_scale, const float *z_p, const float *x_T, const float *eps, const float *x0_q,
                  const float *mu1_q, const float *lv1_q, const float *half_logdet_q, const float *u,
                  float *logratio, int32_t *n_accept, uint32_t *accept_mask, float *mu1_p, float *lv1_p,
                  float *half_logdet_p, float *log_sigma_rows);
/* As csd_resample with x' = mu1_p + exp(lv1_p / 2) * xi and the rejected token's own log Sigma. */
int csd_resample_lv(csd_ctx *ctx, int B, int gamma, int C, int cap, const float *log_sigma_rows,
                    const int32_t *n_accept, const float *mu1_p, const float *lv1_p, const float *mu1_q,
                    const float *lv1_q, const float *xi, const float *v, float *x_new, int32_t *n_prop,
                    uint32_t *flags, int32_t *cap_hits);
/* The three calls above as one round, the two chains concurrent, bit-identical results. */
int csd_round_lv(csd_ctx *ctx, const csd_head *head_q, const csd_head *head_p, const csd_schedule_lv *sched_q,
                 const csd_schedule_lv *sched_p, int B, int gamma, int cfg, float cfg_scale, int cap,
                 const float *z_q, const float *z_p, const float *x_T, const float *eps, const float *u,
                 const float *xi, const float *v, float *x0, float *mu1_q, float *lv1_q, float *half_logdet_q,
                 float *mu1_p, float *lv1_p, float *half_logdet_p, float *log_sigma_rows, float *logratio,
                 int32_t *n_accept, uint32_t *accept_mask, float *x_new, int32_t *n_prop, uint32_t *flags,
                 int32_t *cap_hits);

/* csd_round with the bonus token of the all-accepted branch of Alg. 1 (see csd_verify_bonus): the target chain
 * runs R + B token rows. */
int csd_round_bonus(csd_ctx *ctx, const csd_head *head_q, const csd_head *head_p, const csd_schedule *sched_q,
                    const csd_schedule *sched_p, int B, int gamma, int cfg, float cfg_scale, int cap,
                    const float *z_q, const float *z_p, const float *x_T, const float *eps, const float *u,
                    const float *xi, const float *v, const float *z_next, const float *x_T_next,
                    const float *eps_next, float *x0, float *mu1_q, float *mu1_p, float *logratio,
                    int32_t *n_accept, uint32_t *accept_mask, float *x_new, int32_t *n_prop, uint32_t *flags,
                    int32_t *cap_hits, float *x_bonus, uint32_t *taken);

/* ---- Explicit Gaussian-mixture heads (appendix "More Variants of Diffusion Model", GMM paragraph) ----------
 * With a mixture output head the token distribution p(x) = sum_k pi_k N(x; mu_k, diag(sigma_k^2)) is explicit, so
 * the method needs no diffusion chain: drafts are samples of q, the ratio is p(x)/q(x) itself (accept rule of
 * Sec. 3.1 / Alg. 1), and the modified distribution max(0, p - q)/Z (Eq. 5) is sampled by the same
 * acceptance-rejection loop (Eq. 9-11) with proposals from p: alpha_s = max(0, 1 - q(x')/p(x')).
 * A mixture holds, per token row, K components: logw [rows, K] (unnormalised log-weights, normalised inside),
 * mu and log_sigma [rows, K, C]; all DEVICE arrays, C <= 32.
 *   csd_gmm_draft_sample: x[r] = mu_k + sigma_k * noise[r] with k the first component whose cumulative weight
 *     reaches u_comp[r] in (0,1); comp int32 [R] out or NULL.
 *   csd_gmm_verify: logratio[b,i] = log p(x) - log q(x); accept iff log u <= logratio; n_accept, accept_mask as
 *     csd_verify.  Identical mixtures give exactly 0.
 *   csd_gmm_resample: for sequences with n_accept < gamma, proposals for row b*gamma + n_accept[b]: component from
 *     w[b,k], x' = mu_k + sigma_k * xi[b,k]; outputs as csd_resample (capped loop, flags, cap_hits). */
typedef struct {
  int K;
  const float *logw, *mu, *log_sigma;
} csd_gmm;
int csd_gmm_draft_sample(csd_ctx *ctx, int R, int C, const csd_gmm *q, const float *u_comp, const float *noise,
                         float *x, int32_t *comp);
int csd_gmm_verify(csd_ctx *ctx, int B, int gamma, int C, const csd_gmm *q, const csd_gmm *p, const float *x,
                   const float *u, float *logratio, int32_t *n_accept, uint32_t *accept_mask);
int csd_gmm_resample(csd_ctx *ctx, int B, int gamma, int C, int cap, const csd_gmm *q, const csd_gmm *p,
                     const int32_t *n_accept, const float *w, const float *xi, const float *v, float *x_new,
                     int32_t *n_prop, uint32_t *flags, int32_t *cap_hits);

/* Same computation as csd_round, but every array is a HOST pointer: the call copies the inputs
 * to the device, runs the round, copies the outputs back and synchronises before returning. */
int csd_round_host(csd_ctx *ctx, const csd_head *head_q, const csd_head *head_p,
                   const csd_schedule *sched_q, const csd_schedule *sched_p, int B, int gamma,
                   int cfg, float cfg_scale, int cap, const float *z_q, const float *z_p,
                   const float *x_T, const float *eps, const float *u, const float *xi,
                   const float *v, float *x0, float *mu1_q, float *mu1_p, float *logratio,
                   int32_t *n_accept, uint32_t *accept_mask, float *x_new, int32_t *n_prop,
                   uint32_t *flags, int32_t *cap_hits);

#ifdef __cplusplus
}
#endif
#endif /* CSD_H_ */
