"""Pins of the checker's learned-variance functions (the general Gaussian transition of Eq. 3 with a predicted
diagonal covariance; Sigma of Eq. 7 per token) against closed forms, library densities, the fixed-variance checker
and a statistical law."""
import math

import numpy as np
import pytest
import scipy.stats as st

from oracle import csd_oracle as orc
from paper_2411_11925_b200 import inputs as gen


def _lv_head_weights(spec, rng, const_w=None):
    """A head with 2C outputs.  const_w: make the variance output that constant (zero rows in Wout, bias const_w)."""
    w = gen.make_head_weights(spec, rng)
    C, W = spec.C, spec.W
    bound = math.sqrt(6.0 / (W + 2 * C))
    w["Wout"] = np.concatenate([w["Wout"], rng.uniform(-bound, bound, (C, W)).astype(np.float32)], axis=0)
    w["bout"] = np.concatenate([w["bout"], (0.02 * rng.standard_normal(C)).astype(np.float32)])
    if const_w is not None:
        w["Wout"][C:] = 0.0
        w["bout"][C:] = const_w
    return w


def test_lv_schedule_bounds_are_the_forward_and_the_posterior_variance():
    beta = gen.beta_linear(20, 0.01, 0.3)
    s = orc.lv_schedule(beta, 1.0)
    abar = np.cumprod(1.0 - beta)
    np.testing.assert_allclose(np.exp(s["lv_max"]), beta, rtol=1e-12)
    # posterior variance of x_{t-1} given x_t and a point-mass x_0, by conditioning the joint Gaussian of
    # (x_{t-1}, x_t): var(x_{t-1}) - cov^2 / var(x_t)
    for t in range(2, 21):
        v_prev, v_t = 1.0 - abar[t - 2], 1.0 - abar[t - 1]
        cov = math.sqrt(1.0 - beta[t - 1]) * v_prev
        assert abs(math.exp(s["lv_min"][t - 1]) - (v_prev - cov * cov / v_t)) < 1e-12
    assert s["lv_min"][0] == s["lv_min"][1]                       # the degenerate first step borrows the second's
    assert np.all(s["lv_min"] < s["lv_max"])
    s2 = orc.lv_schedule(beta, 0.8)
    np.testing.assert_allclose(s2["lv_max"] - s["lv_max"], 2 * math.log(0.8), rtol=1e-12)
    np.testing.assert_allclose(s2["lv_min"] - s["lv_min"], 2 * math.log(0.8), rtol=1e-12)
    np.testing.assert_array_equal(s2["a"], s["a"])


@pytest.mark.parametrize("const_w,cfg", [(1.0, False), (1.0, True), (-1.0, False)])
def test_constant_variance_output_reproduces_the_fixed_variance_round(const_w, cfg):
    # w = +1 selects sigma_t^2 = tau^2 beta_t, w = -1 the (clipped) posterior variance: the learned-variance round
    # must then be the fixed-variance round of the same heads with that sigma array, value for value.
    rng = np.random.default_rng(5)
    spec = gen.HeadSpec(2, 128, 64, C=4)
    B, gamma, T, cap, tau = 12, 3, 6, 16, 0.9
    wp = _lv_head_weights(spec, rng, const_w)
    wq = {k: a.copy() for k, a in wp.items()}
    for k in ("W1", "W2", "Wada", "Wout"):                 # close heads: accepts and rejects both occur
        wq[k] = (wp[k] + 3e-4 * rng.standard_normal(wp[k].shape)).astype(np.float32)
    wq["Wout"][spec.C:] = 0.0
    R = B * gamma
    z = rng.standard_normal((R * (2 if cfg else 1), spec.Dz)).astype(np.float32)
    x_T, eps = rng.standard_normal((R, spec.C)), rng.standard_normal((T, R, spec.C))
    u, xi, v = rng.random((B, gamma)), rng.standard_normal((B, cap, spec.C)), rng.random((B, cap))
    beta, tfeat = gen.beta_linear(T, 1e-3, 0.05), gen.timestep_features(T, spec.F)
    lv = orc.lv_schedule(beta, tau)
    got = orc.csd_round_lv(orc.make_mlp_head_lv(wq, z, tfeat, cfg, 2.0), orc.make_mlp_head_lv(wp, z, tfeat, cfg, 2.0),
                           lv, lv, x_T, eps, u, xi, v, B, gamma, cap)
    fixed = orc.ddpm_schedule(beta, tau)
    if const_w < 0:
        fixed = dict(fixed); fixed["sigma"] = np.exp(0.5 * lv["lv_min"])
    cut = lambda w: {**w, "Wout": w["Wout"][:spec.C], "bout": w["bout"][:spec.C]}
    want = orc.csd_round(orc.make_mlp_head(cut(wq), z, tfeat, cfg, 2.0), orc.make_mlp_head(cut(wp), z, tfeat, cfg, 2.0),
                         fixed, fixed, x_T, eps, u, xi, v, B, gamma, cap)
    for k in ("x0", "mu1_q", "mu1_p", "logratio", "x_new"):
        np.testing.assert_allclose(got[k], want[k], rtol=1e-9, atol=1e-9, err_msg=k)
    for k in ("n_accept", "n_prop", "flags"):
        np.testing.assert_array_equal(got[k], want[k], err_msg=k)
    assert 0 < got["n_accept"].sum() < B * gamma
    np.testing.assert_allclose(got["log_sigma_rows"], 0.0, atol=1e-9)      # same variances: Sigma = 1 for every token


def _random_pair(seed=7, cfg=True):
    rng = np.random.default_rng(seed)
    spec_q, spec_p = gen.HeadSpec(1, 128, 64, C=3), gen.HeadSpec(2, 128, 96, C=3)
    B, gamma, T, cap = 5, 4, 7, 8
    R = B * gamma
    wq, wp = _lv_head_weights(spec_q, rng), _lv_head_weights(spec_p, rng)
    rows = R * (2 if cfg else 1)
    zq, zp = rng.standard_normal((rows, 64)).astype(np.float32), rng.standard_normal((rows, 96)).astype(np.float32)
    x_T, eps = rng.standard_normal((R, 3)), rng.standard_normal((T, R, 3))
    u, xi, v = rng.random((B, gamma)), rng.standard_normal((B, cap, 3)), rng.random((B, cap))
    beta, tfeat = gen.beta_linear(T, 1e-3, 0.05), gen.timestep_features(T, 256)
    sq, sp = orc.lv_schedule(beta, 1.0), orc.lv_schedule(beta, 0.95)
    fq, fp = orc.make_mlp_head_lv(wq, zq, tfeat, cfg, 2.5), orc.make_mlp_head_lv(wp, zp, tfeat, cfg, 2.5)
    return fq, fp, sq, sp, x_T, eps, u, xi, v, B, gamma, cap


def test_long_product_equals_per_token_sigma_times_final_step_ratio_with_predicted_variances():
    fq, fp, sq, sp, x_T, eps, u, xi, v, B, gamma, cap = _random_pair()
    out = orc.csd_round_lv(fq, fp, sq, sp, x_T, eps, u, xi, v, B, gamma, cap, keep=True)
    long = orc.log_ratio_long_lv(out["dq"], out["dp"])
    np.testing.assert_allclose(out["logratio"].reshape(-1), long, rtol=1e-9, atol=1e-9)
    # the variances really differ per token, per coordinate and per model
    lv = np.stack(out["dq"]["lvs"])
    assert lv.std(axis=1).min() > 1e-3 and lv.std(axis=2).min() > 1e-4
    assert np.abs(out["log_sigma_rows"]).min() > 1e-3 and out["log_sigma_rows"].std() > 1e-3


def test_aligned_per_step_ratio_is_the_determinant_ratio_of_eq7_by_library_densities():
    # Under shared noise every step t >= 2 contributes sqrt|Sigma_q| / sqrt|Sigma_p| whatever the noise was (Eq. 7):
    # scipy's normal densities at the two recorded paths give that number, and their sum over t >= 2 is the
    # per-token log Sigma; the guided eps_hat and the conditional rows' variance enter as specified.
    fq, fp, sq, sp, x_T, eps, u, xi, v, B, gamma, cap = _random_pair(seed=11)
    out = orc.csd_round_lv(fq, fp, sq, sp, x_T, eps, u, xi, v, B, gamma, cap, keep=True)
    dq, dp = out["dq"], out["dp"]
    T = len(dq["mus"])
    total = 0.0
    for j in range(T - 1):
        t = T - j
        eq_hat, wq = fq(dq["xs"][j], t)
        sd_q = np.exp(0.5 * (sq["lv_min"][t - 1] + 0.5 * (wq + 1) * (sq["lv_max"][t - 1] - sq["lv_min"][t - 1])))
        ep_hat, wp = fp(dp["xs"][j], t)
        sd_p = np.exp(0.5 * (sp["lv_min"][t - 1] + 0.5 * (wp + 1) * (sp["lv_max"][t - 1] - sp["lv_min"][t - 1])))
        lp = st.norm.logpdf(dp["xs"][j + 1], sp["a"][t - 1] * dp["xs"][j] - sp["b"][t - 1] * ep_hat, sd_p).sum(axis=1)
        lq = st.norm.logpdf(dq["xs"][j + 1], sq["a"][t - 1] * dq["xs"][j] - sq["b"][t - 1] * eq_hat, sd_q).sum(axis=1)
        np.testing.assert_allclose(lp - lq, np.log(sd_q).sum(axis=1) - np.log(sd_p).sum(axis=1), rtol=1e-8, atol=1e-8)
        total = total + lp - lq
    np.testing.assert_allclose(out["log_sigma_rows"], total, rtol=1e-9, atol=1e-9)
    # final step: the target scores the draft's x0
    e1, w1 = fp(dp["x1"], 1)
    sd1 = np.exp(0.5 * (sp["lv_min"][0] + 0.5 * (w1 + 1) * (sp["lv_max"][0] - sp["lv_min"][0])))
    lp1 = st.norm.logpdf(out["x0"], sp["a"][0] * dp["x1"] - sp["b"][0] * e1, sd1).sum(axis=1)
    lq1 = st.norm.logpdf(out["x0"], out["mu1_q"], np.exp(0.5 * out["lv1_q"])).sum(axis=1)
    np.testing.assert_allclose(out["logratio"].reshape(-1), total + lp1 - lq1, rtol=1e-9, atol=1e-9)


def test_identical_learned_variance_heads_give_exactly_zero_and_accept_everything():
    fq, fp, sq, sp, x_T, eps, u, xi, v, B, gamma, cap = _random_pair(seed=3)
    out = orc.csd_round_lv(fp, fp, sp, sp, x_T, eps, u, xi, v, B, gamma, cap)
    assert np.all(out["logratio"] == 0.0) and np.all(out["n_accept"] == gamma) and np.all(out["flags"] == 0)


def test_gaussian_logpdf_diag_matches_scipy_multivariate_normal():
    rng = np.random.default_rng(2)
    x, mu, lv = rng.standard_normal((6, 5)), rng.standard_normal((6, 5)), rng.standard_normal((6, 5))
    want = [st.multivariate_normal(mu[i], np.diag(np.exp(lv[i]))).logpdf(x[i]) for i in range(6)]
    np.testing.assert_allclose(orc.gaussian_logpdf_diag(x, mu, lv), want, rtol=1e-12)


def test_resampled_tokens_with_per_dimension_variances_follow_the_normalised_positive_part():
    # C = 2, different variances per coordinate and per model, Sigma != 1: the first coordinate's marginal under
    # max(0, Sigma p - q) / Z, integrated numerically on a grid, against 1e5 draws of the loop (KS), and the mean
    # number of proposals against Sigma / Z.
    N, cap = 100_000, 400
    mu_p, mu_q = np.array([0.0, 0.3]), np.array([0.6, -0.2])
    lv_p, lv_q = np.log(np.array([1.0, 0.49])), np.log(np.array([0.64, 1.21]))
    log_sigma = 0.25
    rng = np.random.default_rng(23)
    xi, v = rng.standard_normal((N, cap, 2)), rng.random((N, cap))
    rep = lambda a: np.broadcast_to(a, (N, 2)).copy()
    out = orc.resample_lv(np.zeros(N, dtype=np.int32), rep(mu_p), rep(lv_p), rep(mu_q), rep(lv_q),
                          np.full(N, log_sigma), xi, v, gamma=1, cap=cap)
    assert out["cap_hits"] == 0
    g0, g1 = np.linspace(-8, 8, 1601), np.linspace(-8, 8, 1601)
    X0, X1 = np.meshgrid(g0, g1, indexing="ij")
    pdf = lambda m, l: st.norm.pdf(X0, m[0], math.exp(0.5 * l[0])) * st.norm.pdf(X1, m[1], math.exp(0.5 * l[1]))
    dens = np.maximum(0.0, math.exp(log_sigma) * pdf(mu_p, lv_p) - pdf(mu_q, lv_q))
    marg = np.trapezoid(dens, g1, axis=1)
    cdf = np.concatenate([[0.0], np.cumsum(0.5 * (marg[1:] + marg[:-1]) * np.diff(g0))])
    Z = cdf[-1]
    res = st.kstest(out["x_new"][:, 0], lambda x: np.interp(x, g0, cdf / Z))
    assert res.pvalue > 1e-3, res
    assert abs(out["n_prop"].mean() - math.exp(log_sigma) / Z) < 0.03 * math.exp(log_sigma) / Z
    # power: draws from p itself fail
    assert st.kstest(rng.normal(mu_p[0], 1.0, N), lambda x: np.interp(x, g0, cdf / Z)).pvalue < 1e-6
