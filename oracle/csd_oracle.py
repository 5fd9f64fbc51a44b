"""Float64 CPU checker for continuous speculative decoding (CSD).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the
method computes, written from the paper; the CUDA library never imports it and
shares no code with it.  Only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may call it.

Everything is numpy float64, vectorised over independent token rows and
otherwise in the paper's order: no blocking, fusion or reordering.

What pins each function (see tests/test_oracle_pins.py):

  ddim_schedule            marginal preservation on Gaussian data for every eta (the sampler's
                           defining property), eta = 1 on the full ladder is the DDPM posterior,
                           last-step mean is x0_hat
  ddpm_schedule            textbook special case (N(0,1) data: mu_t = sqrt(alpha_t) x_t)
  denoise / run_pair       Theorem 1 pathwise identity and its Monte-Carlo form
  log_sigma_term, log_ratio_*   long form (Eq. 4) == closed form (Eq. 7, 8);
                           identical heads give exactly 0; 1-D Gaussian toy
                           head matches an independently composed affine map
  log_ratio_single_path    T = 1 reduces to Eq. 8; identical heads give exactly 0;
                           1-D Gaussian toy heads: equals the difference of two
                           multivariate-normal log-densities of the whole path
                           (library routine); E_q[p(Y)/q(Y)] = 1 by Monte Carlo
  lv_schedule, denoise_lv, log_ratio_*_lv, resample_lv, csd_round_lv (learned diagonal variances)
                           a head whose variance output is the constant +1 reproduces the fixed-variance
                           round exactly; long form (Eq. 4) == closed form (Eq. 7, 8) per token; 1-D toy
                           heads against scipy's normal densities over the whole pair of paths; posterior
                           variance against the textbook closed form; KS of the resampler with different
                           per-dimension variances against the numerically integrated max(0, Sigma p - q)
  gmm_logpdf, gmm_sample, gmm_resample, gmm_round (explicit mixture heads)
                           scipy's multivariate-normal densities and logsumexp; one component reduces to the
                           diagonal Gaussian; KS of the draws against the mixture CDF and of the resampled tokens
                           against the numerically integrated max(0, p - q); acceptance rate = 1 - TV(p, q)
  accept_prefix            brute force over all accept masks (Alg. 1)
  resample                 KS test against the numerically integrated
                           max(0, Sigma*p - q) (Eq. 5, Eq. 11, Cor. 1); textbook
                           total-variation acceptance rate
  silu, layer_norm, timestep MLP   library routines (torch float64)
  head_eps (architecture)  PARITY UNPINNED by the paper: the paper does not
                           describe the diffusion head; its layout is this
                           project's own specification.  Only structural
                           special cases are pinned.
"""
from __future__ import annotations

from typing import Callable, Dict, Optional, Tuple

import numpy as np

f64 = np.float64


# --------------------------------------------------------------------------
# Noise schedule: the Gaussian transition of Eq. 3, N(x_{t-1}; mu, Sigma), with
# the epsilon-prediction mean of the DDPM work the paper cites for Eq. 3 and a
# fixed isotropic variance sigma_t^2 = tau^2 * beta_t (temperature, Appendix
# "Temperature").
# --------------------------------------------------------------------------
def ddpm_schedule(beta: np.ndarray, tau: float = 1.0) -> Dict[str, np.ndarray]:
    beta = np.asarray(beta, dtype=f64)
    alpha = 1.0 - beta
    alphabar = np.cumprod(alpha)
    a = 1.0 / np.sqrt(alpha)                              # mu_t = a_t x_t - b_t eps_hat
    b = beta / (np.sqrt(alpha) * np.sqrt(1.0 - alphabar))
    sigma = tau * np.sqrt(beta)
    return {"a": a, "b": b, "sigma": sigma, "alphabar": alphabar, "beta": beta}


def ddim_schedule(beta_full: np.ndarray, steps: np.ndarray, eta: float) -> Dict[str, np.ndarray]:
    """DDIM sampler (Appendix "More Variants of Diffusion Model") derived from a DDPM trained with beta_full,
    run on the ascending sub-sequence `steps` (1-based timesteps) with stochasticity eta in (0, 1].  The
    transition is the Gaussian q_sigma(x_prev | x_t, x0_hat) of the DDIM paper:
      x0_hat = (x_t - sqrt(1-ab_t) eps_hat) / sqrt(ab_t)
      x_prev = sqrt(ab_prev) x0_hat + sqrt(1 - ab_prev - sigma^2) eps_hat + sigma eps,
      sigma  = eta sqrt((1-ab_prev)/(1-ab_t)) sqrt(1 - ab_t/ab_prev),
    i.e. mean a x_t - b eps_hat, so it enters the method exactly like Eq. 3.  At the last step ab_prev = 1 makes
    sigma = 0, a point mass that has no density ratio: there sigma = eta sqrt(1 - ab_t) (the variance of the
    respaced chain's forward step), mean x0_hat.  Index k-1 of the result is the k-th step counted from x_0."""
    ab_full = np.cumprod(1.0 - np.asarray(beta_full, dtype=f64))
    steps = np.asarray(steps, dtype=np.int64)
    ab = ab_full[steps - 1]
    ab_prev = np.concatenate([[1.0], ab[:-1]])
    sigma = eta * np.sqrt((1.0 - ab_prev) / (1.0 - ab)) * np.sqrt(1.0 - ab / ab_prev)
    sigma[0] = eta * np.sqrt(1.0 - ab[0])
    direction = np.sqrt(np.maximum(0.0, 1.0 - ab_prev - sigma ** 2))
    direction[0] = 0.0
    a = np.sqrt(ab_prev / ab)
    b = a * np.sqrt(1.0 - ab) - direction
    return {"a": a, "b": b, "sigma": sigma, "alphabar": ab, "beta": 1.0 - ab / ab_prev}


# --------------------------------------------------------------------------
# The per-token diffusion head eps_hat = head(x_t, t, z) (the "diffusion loss"
# module of Sec. "Implementation Details"; architecture = project spec).
# --------------------------------------------------------------------------
def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def layer_norm(h: np.ndarray, eps: float = 1e-6) -> np.ndarray:
    """No affine parameters, biased variance over the last axis."""
    m = h.mean(axis=-1, keepdims=True)
    v = ((h - m) ** 2).mean(axis=-1, keepdims=True)
    return (h - m) / np.sqrt(v + eps)


def timestep_embedding(w: Dict[str, np.ndarray], tfeat_t: np.ndarray) -> np.ndarray:
    """te_t = Wt2 SiLU(Wt1 tfeat_t + bt1) + bt2, one vector of width W."""
    hid = silu(np.asarray(w["Wt1"], dtype=f64) @ tfeat_t.astype(f64) + np.asarray(w["bt1"], dtype=f64))
    return np.asarray(w["Wt2"], dtype=f64) @ hid + np.asarray(w["bt2"], dtype=f64)


def head_eps(w: Dict[str, np.ndarray], x_t: np.ndarray, tfeat_t: np.ndarray, z: np.ndarray,
             trace: Optional[dict] = None) -> np.ndarray:
    """eps_hat for a batch of head rows.  x_t [N,C], z [N,Dz], tfeat_t [F]."""
    W64 = {k: np.asarray(v, dtype=f64) for k, v in w.items()}   # no copy when already float64
    x_t = x_t.astype(f64)
    cz = z.astype(f64) @ W64["Wz"].T + W64["bz"]
    te = timestep_embedding(w, tfeat_t)
    s = silu(cz + te[None, :])
    h = x_t @ W64["Win"].T + W64["bin"]
    L = W64["W1"].shape[0]
    Wd = W64["W1"].shape[1]
    if trace is not None:
        trace["s"] = s.copy(); trace["h_in"] = h.copy(); trace["h"] = []
    for k in range(L):
        mod = s @ W64["Wada"][k].T + W64["bada"][k]
        shift, scale, gate = mod[:, :Wd], mod[:, Wd:2 * Wd], mod[:, 2 * Wd:]
        u = layer_norm(h) * (1.0 + scale) + shift
        u = silu(u @ W64["W1"][k].T + W64["b1"][k])
        u = u @ W64["W2"][k].T + W64["b2"][k]
        h = h + gate * u
        if trace is not None:
            trace["h"].append(h.copy())
    mod = s @ W64["Wfada"].T + W64["bfada"]
    shift, scale = mod[:, :Wd], mod[:, Wd:]
    uf = layer_norm(h) * (1.0 + scale) + shift
    return uf @ W64["Wout"].T + W64["bout"]


def make_mlp_head(w: Dict[str, np.ndarray], z: np.ndarray, tfeat: np.ndarray,
                  cfg: bool, cfg_scale: float) -> Callable[[np.ndarray, int], np.ndarray]:
    """Return eps_fn(x_t [R,C], t) with classifier-free guidance folded in:
    rows [0,R) of z are conditional, rows [R,2R) unconditional, both halves see
    the same x_t, and eps = eps_u + scale*(eps_c - eps_u) (Appendix
    "Classifier-Free Guidance")."""
    w = {k: np.asarray(v, dtype=f64) for k, v in w.items()}   # widen once, not at every step

    def eps_fn(x_t: np.ndarray, t: int) -> np.ndarray:
        R = x_t.shape[0]
        if cfg:
            e = head_eps(w, np.concatenate([x_t, x_t], axis=0), tfeat[t - 1], z)
            e_c, e_u = e[:R], e[R:]
            return e_u + cfg_scale * (e_c - e_u)
        return head_eps(w, x_t, tfeat[t - 1], z)
    return eps_fn


def make_gaussian_toy_head(m: float, s: float, alphabar: np.ndarray
                           ) -> Callable[[np.ndarray, int], np.ndarray]:
    """Analytic eps-predictor when the data are N(m, s^2) per coordinate:
    x_t ~ N(sqrt(ab) m, ab s^2 + 1 - ab) and
    E[eps | x_t] = sqrt(1-ab) (x_t - sqrt(ab) m) / (ab s^2 + 1 - ab)."""
    def eps_fn(x_t: np.ndarray, t: int) -> np.ndarray:
        ab = alphabar[t - 1]
        return np.sqrt(1.0 - ab) * (x_t - np.sqrt(ab) * m) / (ab * s * s + 1.0 - ab)
    return eps_fn


# --------------------------------------------------------------------------
# Denoising trajectories (Eq. 1, Eq. 3; reparameterised sampling
# x_{t-1} = sqrt(Sigma) eps_t + mu, Sec. 3.2 / Appendix A.2)
# --------------------------------------------------------------------------
def denoise(eps_fn: Callable[[np.ndarray, int], np.ndarray], sched: Dict[str, np.ndarray],
            x_T: np.ndarray, noise: np.ndarray, sample_last: bool = True,
            keep: bool = False) -> Dict[str, np.ndarray]:
    """Run t = T..1.  noise[t-1] is the N(0,I) draw of step t.  Noise is added at
    every step including t=1, because p(x_0|x_1) must be a proper Gaussian to take
    ratios of (Eq. 8) and to propose from (Cor. 1).  With sample_last=False the
    last step only yields mu_1 (the target never samples x_0: it evaluates the
    density of the draft's x_0, Appendix A.2 after the ratio derivation)."""
    T = len(sched["a"])
    x = x_T.astype(f64)
    xs = [x.copy()] if keep else None       # xs[j] = x_{T-j}
    mus = [] if keep else None              # mus[j] = mu_{T-j}
    x1 = mu1 = x0 = None
    for t in range(T, 0, -1):
        e_hat = eps_fn(x, t)
        mu = sched["a"][t - 1] * x - sched["b"][t - 1] * e_hat
        if t == 1:
            x1, mu1 = x, mu
        if t > 1 or sample_last:
            x = mu + sched["sigma"][t - 1] * noise[t - 1].astype(f64)
            if t == 1:
                x0 = x
        if keep:
            mus.append(mu.copy())
            if t > 1 or sample_last:
                xs.append(x.copy())
    out = {"x1": x1, "mu1": mu1, "x0": x0}
    if keep:
        out["xs"], out["mus"] = xs, mus
    return out


def run_pair(eps_q, eps_p, sched_q, sched_p, x_T, noise, noise_p=None, keep=False):
    """Draft and target trajectories from the same x_T (Eq. 8 assumes
    p(x_T^p) = q(x_T^q)).  Denoising trajectory alignment = both use the same
    noise; pass noise_p to break the alignment (ablation of Table 6)."""
    dq = denoise(eps_q, sched_q, x_T, noise, sample_last=True, keep=keep)
    dp = denoise(eps_p, sched_p, x_T, noise if noise_p is None else noise_p,
                 sample_last=False, keep=keep)
    return dq, dp


# --------------------------------------------------------------------------
# Ratio of joint path densities (Eq. 4), its alignment simplification (Eq. 7, 8)
# --------------------------------------------------------------------------
def gaussian_logpdf_iso(x: np.ndarray, mu: np.ndarray, sigma: float) -> np.ndarray:
    """log N(x; mu, sigma^2 I) over the last axis (standard form, with the minus
    sign the paper's printed density dropped)."""
    C = x.shape[-1]
    d = x - mu
    return (-0.5 * C * np.log(2.0 * np.pi) - C * np.log(sigma)
            - 0.5 * np.sum(d * d, axis=-1) / (sigma * sigma))


def log_sigma_term(sigma_q: np.ndarray, sigma_p: np.ndarray, C: int) -> float:
    """log of Sigma = prod_{t=2..T} sqrt|Sigma_q,t| / sqrt|Sigma_p,t| (Eq. 7) for
    isotropic variances: C * sum_{t>=2} (log sigma_q,t - log sigma_p,t)."""
    return float(C * np.sum(np.log(sigma_q[1:]) - np.log(sigma_p[1:])))


def log_ratio_closed(x0, mu1_q, mu1_p, sigma1_q, sigma1_p, log_sigma) -> np.ndarray:
    """log [ Sigma * p(x_0 | x_1^p) / q(x_0 | x_1^q) ]  (Eq. 8)."""
    return (log_sigma + gaussian_logpdf_iso(x0, mu1_p, sigma1_p)
            - gaussian_logpdf_iso(x0, mu1_q, sigma1_q))


def log_ratio_long(dq: dict, dp: dict, sched_q, sched_p) -> np.ndarray:
    """log p(Y_p)/q(Y_q) as the full product over t = 1..T of per-step Gaussian
    ratios (Eq. 4) with x_0^p := x_0^q, p(x_T) = q(x_T).  Needs keep=True runs."""
    T = len(sched_q["a"])
    total = 0.0
    for j in range(T):                       # j-th step handles t = T-j
        t = T - j
        xq_next = dq["xs"][j + 1]
        xp_next = dp["xs"][j + 1] if t > 1 else dq["xs"][j + 1]
        total = total + gaussian_logpdf_iso(xp_next, dp["mus"][j], sched_p["sigma"][t - 1]) \
                      - gaussian_logpdf_iso(xq_next, dq["mus"][j], sched_q["sigma"][t - 1])
    return total


def log_ratio_single_path(eps_p: Callable[[np.ndarray, int], np.ndarray], sched_q, sched_p,
                          dq: dict) -> np.ndarray:
    """log p(Y_q)/q(Y_q) of Eq. 2: the exact criterion, in which BOTH models score the
    draft's own trajectory Y_q = (x_T, x^q_{T-1}, ..., x^q_0).  Step t contributes
    log N(x^q_{t-1}; mu^p_t(x^q_t), sigma_p,t^2) - log N(x^q_{t-1}; mu^q_t(x^q_t), sigma_q,t^2);
    p(x_T) = q(x_T) cancels.  dq is a keep=True draft run: xs[j] = x^q_{T-j}, mus[j] = mu^q_{T-j}."""
    T = len(sched_q["a"])
    total = 0.0
    for j in range(T):
        t = T - j
        x_t, x_next = dq["xs"][j], dq["xs"][j + 1]
        mu_p = sched_p["a"][t - 1] * x_t - sched_p["b"][t - 1] * eps_p(x_t, t)
        total = total + gaussian_logpdf_iso(x_next, mu_p, sched_p["sigma"][t - 1]) \
                      - gaussian_logpdf_iso(x_next, dq["mus"][j], sched_q["sigma"][t - 1])
    return total


# --------------------------------------------------------------------------
# Verification (Alg. 1: draw r_i, accept while r_i <= ratio, n = first reject)
# --------------------------------------------------------------------------
def accept_prefix(log_ratio: np.ndarray, u: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """log_ratio, u: [B, gamma].  Position i is rejected iff u > p/q (so it is
    accepted iff log u <= log ratio); n[b] = number of leading accepts."""
    acc = np.log(u.astype(f64)) <= log_ratio
    B, g = acc.shape
    n = np.full(B, g, dtype=np.int32)
    for b in range(B):
        for i in range(g):
            if not acc[b, i]:
                n[b] = i
                break
    return n, acc


# --------------------------------------------------------------------------
# Resampling from the modified distribution max(0, p - q)/Z (Eq. 5) by
# acceptance-rejection with bound M = 1/Z (Eq. 9-11) in the form of Corollary 1:
# propose x' ~ p(x_0 | x_1^p), accept with
#   alpha_s = max(0, Sigma p(x'|x_1^p) - q(x'|x_1^q)) / (Sigma p(x'|x_1^p)).
# --------------------------------------------------------------------------
def resample(n_accept, mu1_p, mu1_q, sigma1_p, sigma1_q, log_sigma, xi, v, gamma, cap):
    B = len(n_accept)
    C = mu1_p.shape[-1]
    x_new = np.zeros((B, C), dtype=f64)
    n_prop = np.zeros(B, dtype=np.int32)
    flags = np.zeros(B, dtype=np.uint32)
    alpha_first = np.full(B, np.nan)
    for b in range(B):
        n = int(n_accept[b])
        if n >= gamma:
            continue                          # all accepted: nothing to resample
        j = b * gamma + n                     # first rejected position
        flags[b] |= 1
        done = False
        for k in range(cap):
            xp = mu1_p[j] + sigma1_p * xi[b, k].astype(f64)
            lp = gaussian_logpdf_iso(xp, mu1_p[j], sigma1_p)
            lq = gaussian_logpdf_iso(xp, mu1_q[j], sigma1_q)
            # alpha_s = max(0, 1 - q/(Sigma p)), evaluated in the log domain
            alpha_s = max(0.0, -np.expm1(min(0.0, lq - log_sigma - lp)))
            if k == 0:
                alpha_first[b] = alpha_s
            x_new[b] = xp
            n_prop[b] = k + 1
            if float(v[b, k]) <= alpha_s:
                done = True
                break
        if not done:
            flags[b] |= 2                     # cap hit: last proposal is returned
    return {"x_new": x_new, "n_prop": n_prop, "flags": flags,
            "cap_hits": int(np.sum((flags & 2) != 0)), "alpha_first": alpha_first}


# --------------------------------------------------------------------------
# One full speculative round (Alg. 1 without the AR backbones)
# --------------------------------------------------------------------------
def csd_round(eps_q, eps_p, sched_q, sched_p, x_T, noise, u, xi, v, B, gamma, cap,
              keep=False) -> Dict[str, np.ndarray]:
    C = x_T.shape[-1]
    dq, dp = run_pair(eps_q, eps_p, sched_q, sched_p, x_T, noise, keep=keep)
    ls = log_sigma_term(sched_q["sigma"], sched_p["sigma"], C)
    s1q, s1p = sched_q["sigma"][0], sched_p["sigma"][0]
    logr = log_ratio_closed(dq["x0"], dq["mu1"], dp["mu1"], s1q, s1p, ls)
    n, acc = accept_prefix(logr.reshape(B, gamma), u)
    rs = resample(n, dp["mu1"], dq["mu1"], s1p, s1q, ls, xi, v, gamma, cap)
    out = {"x0": dq["x0"], "mu1_q": dq["mu1"], "x1_q": dq["x1"], "mu1_p": dp["mu1"],
           "x1_p": dp["x1"], "log_sigma": ls, "logratio": logr.reshape(B, gamma),
           "n_accept": n, "accept": acc, **rs}
    if keep:
        out["dq"], out["dp"] = dq, dp
    return out


def bonus_token(eps_p_next, sched_p, x_T_next, noise_next, n_accept, gamma) -> Dict[str, np.ndarray]:
    """Alg. 1, all-accepted branch: a sequence whose gamma drafts were all accepted also gets the token of
    position gamma+1, an ordinary sample x_0 of the target head's reverse process at that position (noise at every
    step, as for the draft).  Rows of other sequences are left at zero with taken = False."""
    d = denoise(eps_p_next, sched_p, x_T_next, noise_next, sample_last=True)
    taken = np.asarray(n_accept) >= gamma
    x = np.where(taken[:, None], d["x0"], 0.0)
    return {"x_bonus": x, "taken": taken, "x0_all": d["x0"]}


def single_path_from_inputs(inp) -> Dict[str, np.ndarray]:
    """Draft trajectories of a RoundInputs bundle and the exact ratio of Eq. 2 on them,
    with the accept scan of Alg. 1 applied to that ratio."""
    wl = inp.wl
    sched = ddpm_schedule(inp.beta, wl.tau)
    eq = make_mlp_head(inp.w_q, inp.z_q, inp.tfeat, wl.cfg, wl.cfg_scale)
    ep = make_mlp_head(inp.w_p, inp.z_p, inp.tfeat, wl.cfg, wl.cfg_scale)
    dq = denoise(eq, sched, inp.x_T, inp.eps, sample_last=True, keep=True)
    logr = log_ratio_single_path(ep, sched, sched, dq).reshape(wl.B, wl.gamma)
    n, acc = accept_prefix(logr, inp.u)
    return {"traj_x": np.stack(dq["xs"]), "traj_mu": np.stack(dq["mus"]), "logratio": logr,
            "n_accept": n, "accept": acc}


def round_from_inputs(inp, keep: bool = False) -> Dict[str, np.ndarray]:
    """Run csd_round on a RoundInputs bundle (MLP heads, linear-beta schedule)."""
    wl = inp.wl
    sched = ddpm_schedule(inp.beta, wl.tau)
    eq = make_mlp_head(inp.w_q, inp.z_q, inp.tfeat, wl.cfg, wl.cfg_scale)
    ep = make_mlp_head(inp.w_p, inp.z_p, inp.tfeat, wl.cfg, wl.cfg_scale)
    return csd_round(eq, ep, sched, sched, inp.x_T, inp.eps, inp.u, inp.xi, inp.v,
                     wl.B, wl.gamma, wl.cap, keep=keep)


# --------------------------------------------------------------------------
# Learned per-dimension variances: the general transition of Eq. 3,
# N(x_{t-1}; mu_theta(x_t, t), Sigma_theta(x_t, t)) with a diagonal Sigma_theta that the head predicts
# next to eps_hat (the paper cites the improved-DDPM work for this network).  The head then has 2C
# outputs [eps_hat | w]; the log-variance of coordinate d interpolates, with f = (w_d + 1) / 2, between
# two per-step bounds:   log var_{t,d} = lv_min[t] + f * (lv_max[t] - lv_min[t]).
# lv_schedule gives the bounds of that work for a DDPM: lv_max = log beta_t, lv_min = log of the
# posterior variance beta~_t = beta_t (1 - abar_{t-1}) / (1 - abar_t), with beta~_1 (= 0) replaced by
# beta~_2; a temperature tau scales both standard deviations (adds 2 log tau).
# --------------------------------------------------------------------------
def lv_schedule(beta: np.ndarray, tau: float = 1.0) -> Dict[str, np.ndarray]:
    s = ddpm_schedule(beta, 1.0)
    abar = s["alphabar"]
    abar_prev = np.concatenate([[1.0], abar[:-1]])
    post = s["beta"] * (1.0 - abar_prev) / (1.0 - abar)
    if len(post) > 1:
        post[0] = post[1]
    else:
        post[0] = s["beta"][0]
    return {"a": s["a"], "b": s["b"], "lv_min": np.log(post) + 2.0 * np.log(tau),
            "lv_max": np.log(s["beta"]) + 2.0 * np.log(tau), "alphabar": abar, "beta": s["beta"]}


def make_mlp_head_lv(w: Dict[str, np.ndarray], z: np.ndarray, tfeat: np.ndarray, cfg: bool, cfg_scale: float):
    """Head with 2C outputs: returns fn(x_t [R,C], t) -> (eps_hat [R,C], w [R,C]).  With classifier-free
    guidance eps_hat is guided as in make_mlp_head; the variance output is the conditional row's own
    (guidance acts on the predicted noise only)."""
    w = {k: np.asarray(v, dtype=f64) for k, v in w.items()}

    def fn(x_t: np.ndarray, t: int):
        R, C = x_t.shape
        if cfg:
            o = head_eps(w, np.concatenate([x_t, x_t], axis=0), tfeat[t - 1], z)
            e_c, e_u = o[:R, :C], o[R:, :C]
            return e_u + cfg_scale * (e_c - e_u), o[:R, C:]
        o = head_eps(w, x_t, tfeat[t - 1], z)
        return o[:, :C], o[:, C:]
    return fn


def denoise_lv(fn, sched: Dict[str, np.ndarray], x_T: np.ndarray, noise: np.ndarray, sample_last: bool = True,
               keep: bool = False) -> Dict[str, np.ndarray]:
    """As denoise(), with the transition's diagonal variance predicted at every step:
    x_{t-1} = mu_t + exp(lv_t / 2) * noise_t.  Returns also lv1 (log-variance of the last step, [R,C]) and
    half_logdet = (1/2) sum_{t>=2} sum_d lv_{t,d}, i.e. log prod_{t>=2} sqrt|Sigma_t| of this trajectory."""
    T = len(sched["a"])
    x = x_T.astype(f64)
    xs = [x.copy()] if keep else None
    mus, lvs = ([] if keep else None), ([] if keep else None)
    half_logdet = np.zeros(x.shape[0], dtype=f64)
    x1 = mu1 = x0 = lv1 = None
    for t in range(T, 0, -1):
        e_hat, wv = fn(x, t)
        lv = sched["lv_min"][t - 1] + 0.5 * (wv + 1.0) * (sched["lv_max"][t - 1] - sched["lv_min"][t - 1])
        mu = sched["a"][t - 1] * x - sched["b"][t - 1] * e_hat
        if t == 1:
            x1, mu1, lv1 = x, mu, lv
        else:
            half_logdet = half_logdet + 0.5 * np.sum(lv, axis=-1)
        if t > 1 or sample_last:
            x = mu + np.exp(0.5 * lv) * noise[t - 1].astype(f64)
            if t == 1:
                x0 = x
        if keep:
            mus.append(mu.copy()); lvs.append(lv.copy())
            if t > 1 or sample_last:
                xs.append(x.copy())
    out = {"x1": x1, "mu1": mu1, "x0": x0, "lv1": lv1, "half_logdet": half_logdet}
    if keep:
        out["xs"], out["mus"], out["lvs"] = xs, mus, lvs
    return out


def gaussian_logpdf_diag(x: np.ndarray, mu: np.ndarray, lv: np.ndarray) -> np.ndarray:
    """log N(x; mu, diag(exp(lv))) over the last axis."""
    C = x.shape[-1]
    d = x - mu
    return -0.5 * C * np.log(2.0 * np.pi) - 0.5 * np.sum(lv, axis=-1) - 0.5 * np.sum(d * d * np.exp(-lv), axis=-1)


def log_ratio_closed_lv(x0, mu1_q, lv1_q, mu1_p, lv1_p, log_sigma_rows) -> np.ndarray:
    """Eq. 8 with Sigma of Eq. 7 per token: log Sigma[r] = half_logdet_q[r] - half_logdet_p[r]."""
    return log_sigma_rows + gaussian_logpdf_diag(x0, mu1_p, lv1_p) - gaussian_logpdf_diag(x0, mu1_q, lv1_q)


def log_ratio_long_lv(dq: dict, dp: dict) -> np.ndarray:
    """The full product of Eq. 4 over t = 1..T with x_0^p := x_0^q (keep=True runs of denoise_lv)."""
    T = len(dq["mus"])
    total = 0.0
    for j in range(T):
        t = T - j
        xp_next = dp["xs"][j + 1] if t > 1 else dq["xs"][j + 1]
        total = total + gaussian_logpdf_diag(xp_next, dp["mus"][j], dp["lvs"][j]) \
                      - gaussian_logpdf_diag(dq["xs"][j + 1], dq["mus"][j], dq["lvs"][j])
    return total


def resample_lv(n_accept, mu1_p, lv1_p, mu1_q, lv1_q, log_sigma_rows, xi, v, gamma, cap):
    """Corollary 1 with diagonal final-step covariances: propose x' = mu_p + exp(lv_p / 2) xi, accept with
    alpha_s = max(0, 1 - q(x') / (Sigma p(x'))), Sigma the rejected token's own (Eq. 7)."""
    B = len(n_accept)
    C = mu1_p.shape[-1]
    x_new = np.zeros((B, C), dtype=f64)
    n_prop = np.zeros(B, dtype=np.int32)
    flags = np.zeros(B, dtype=np.uint32)
    for b in range(B):
        n = int(n_accept[b])
        if n >= gamma:
            continue
        j = b * gamma + n
        flags[b] |= 1
        done = False
        for k in range(cap):
            xp = mu1_p[j] + np.exp(0.5 * lv1_p[j]) * xi[b, k].astype(f64)
            lp = gaussian_logpdf_diag(xp, mu1_p[j], lv1_p[j])
            lq = gaussian_logpdf_diag(xp, mu1_q[j], lv1_q[j])
            alpha_s = max(0.0, -np.expm1(min(0.0, lq - log_sigma_rows[j] - lp)))
            x_new[b] = xp
            n_prop[b] = k + 1
            if float(v[b, k]) <= alpha_s:
                done = True
                break
        if not done:
            flags[b] |= 2
    return {"x_new": x_new, "n_prop": n_prop, "flags": flags, "cap_hits": int(np.sum((flags & 2) != 0))}


def csd_round_lv(fn_q, fn_p, sched_q, sched_p, x_T, noise, u, xi, v, B, gamma, cap, keep=False):
    """One round of Alg. 1 with heads that predict their variances."""
    dq = denoise_lv(fn_q, sched_q, x_T, noise, sample_last=True, keep=keep)
    dp = denoise_lv(fn_p, sched_p, x_T, noise, sample_last=False, keep=keep)
    ls = dq["half_logdet"] - dp["half_logdet"]
    logr = log_ratio_closed_lv(dq["x0"], dq["mu1"], dq["lv1"], dp["mu1"], dp["lv1"], ls)
    n, acc = accept_prefix(logr.reshape(B, gamma), u)
    rs = resample_lv(n, dp["mu1"], dp["lv1"], dq["mu1"], dq["lv1"], ls, xi, v, gamma, cap)
    out = {"x0": dq["x0"], "mu1_q": dq["mu1"], "lv1_q": dq["lv1"], "x1_q": dq["x1"], "mu1_p": dp["mu1"],
           "lv1_p": dp["lv1"], "half_logdet_q": dq["half_logdet"], "half_logdet_p": dp["half_logdet"],
           "log_sigma_rows": ls, "logratio": logr.reshape(B, gamma), "n_accept": n, "accept": acc, **rs}
    if keep:
        out["dq"], out["dp"] = dq, dp
    return out


# --------------------------------------------------------------------------
# Gaussian-mixture output heads (Appendix "More Variants of Diffusion Model"): the AR model emits, per token, an
# explicit mixture p(x) = sum_k pi_k N(x; mu_k, diag(sigma_k^2)) instead of a diffusion head.  Both densities are
# then available in closed form, so the accept test is the plain rule of Sec. 3.1 (accept iff u <= p(x)/q(x)) and the
# modified distribution max(0, p - q)/Z (Eq. 5) is sampled by the same acceptance-rejection loop (Eq. 9-11) with
# proposals from p itself: alpha_s = max(0, p(x') - q(x')) / p(x').
# A mixture is (logw [N,K] unnormalised log-weights, mu [N,K,C], log_sigma [N,K,C]).
# --------------------------------------------------------------------------
def _logsumexp(a: np.ndarray, axis: int) -> np.ndarray:
    m = np.max(a, axis=axis, keepdims=True)
    return np.squeeze(m, axis=axis) + np.log(np.sum(np.exp(a - m), axis=axis))


def gmm_logpdf(x: np.ndarray, logw: np.ndarray, mu: np.ndarray, log_sigma: np.ndarray) -> np.ndarray:
    x, logw, mu, log_sigma = (np.asarray(a, dtype=f64) for a in (x, logw, mu, log_sigma))
    C = x.shape[-1]
    lw = logw - _logsumexp(logw, axis=-1)[..., None]
    t = (x[:, None, :] - mu) * np.exp(-log_sigma)
    comp = lw - np.sum(log_sigma, axis=-1) - 0.5 * np.sum(t * t, axis=-1) - 0.5 * C * np.log(2.0 * np.pi)
    return _logsumexp(comp, axis=-1)


def gmm_sample(logw, mu, log_sigma, u_comp, noise) -> Tuple[np.ndarray, np.ndarray]:
    """x = mu_k + sigma_k * noise with k drawn by inverting the weights' CDF at u_comp: the first k whose cumulative
    weight reaches u_comp (the last component if rounding leaves the total short of it)."""
    logw, mu, log_sigma = (np.asarray(a, dtype=f64) for a in (logw, mu, log_sigma))
    w = np.exp(logw - _logsumexp(logw, axis=-1)[..., None])
    cum = np.cumsum(w, axis=-1)
    K = w.shape[-1]
    comp = np.minimum((cum < np.asarray(u_comp, dtype=f64)[:, None]).sum(axis=-1), K - 1).astype(np.int32)
    rows = np.arange(len(comp))
    x = mu[rows, comp] + np.exp(log_sigma[rows, comp]) * np.asarray(noise, dtype=f64)
    return x, comp


def gmm_resample(n_accept, q, p, w, xi, v, gamma, cap):
    """q, p: mixtures (logw, mu, log_sigma) over the R = B gamma token rows; proposals x' ~ p of the first rejected
    row (component from w[b,k], Gaussian draw xi[b,k]), consumed in order, accepted iff v <= max(0, 1 - q(x')/p(x'))."""
    B = len(n_accept)
    C = p[1].shape[-1]
    x_new = np.zeros((B, C), dtype=f64)
    n_prop = np.zeros(B, dtype=np.int32)
    flags = np.zeros(B, dtype=np.uint32)
    for b in range(B):
        n = int(n_accept[b])
        if n >= gamma:
            continue
        j = b * gamma + n
        flags[b] |= 1
        done = False
        pj = tuple(a[j:j + 1] for a in p)
        qj = tuple(a[j:j + 1] for a in q)
        for k in range(cap):
            xp, _ = gmm_sample(pj[0], pj[1], pj[2], np.array([w[b, k]]), xi[b, k][None, :])
            lp, lq = gmm_logpdf(xp, *pj)[0], gmm_logpdf(xp, *qj)[0]
            alpha_s = max(0.0, -np.expm1(min(0.0, lq - lp)))
            x_new[b] = xp[0]
            n_prop[b] = k + 1
            if float(v[b, k]) <= alpha_s:
                done = True
                break
        if not done:
            flags[b] |= 2
    return {"x_new": x_new, "n_prop": n_prop, "flags": flags, "cap_hits": int(np.sum((flags & 2) != 0))}


def gmm_round(q, p, u_comp, noise, u, w, xi, v, B, gamma, cap) -> Dict[str, np.ndarray]:
    """One round of Alg. 1 with explicit mixture heads: drafts x_i ~ q_i, ratio p_i(x_i)/q_i(x_i), accepted prefix,
    resampling of the first rejected position from max(0, p - q)/Z."""
    x, comp = gmm_sample(q[0], q[1], q[2], u_comp, noise)
    logr = gmm_logpdf(x, *p) - gmm_logpdf(x, *q)
    n, acc = accept_prefix(logr.reshape(B, gamma), u)
    rs = gmm_resample(n, q, p, w, xi, v, gamma, cap)
    return {"x": x, "comp": comp, "logratio": logr.reshape(B, gamma), "n_accept": n, "accept": acc, **rs}
