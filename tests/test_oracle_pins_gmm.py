"""Pins of the checker's Gaussian-mixture functions (explicit output distributions, appendix on model variants)."""
import math

import numpy as np
import scipy.special as sp
import scipy.stats as st

from oracle import csd_oracle as orc


def _mix(rng, N, K, C, spread=1.0):
    return (rng.standard_normal((N, K)), spread * rng.standard_normal((N, K, C)), 0.3 * rng.standard_normal((N, K, C)) - 0.5)


def test_gmm_logpdf_matches_scipy_mixture_and_single_component_is_the_diagonal_gaussian():
    rng = np.random.default_rng(1)
    N, K, C = 7, 5, 3
    logw, mu, ls = _mix(rng, N, K, C)
    x = rng.standard_normal((N, C))
    got = orc.gmm_logpdf(x, logw, mu, ls)
    pi = sp.softmax(logw, axis=1)
    for i in range(N):
        dens = sum(pi[i, k] * st.multivariate_normal(mu[i, k], np.diag(np.exp(2 * ls[i, k]))).pdf(x[i]) for k in range(K))
        assert abs(got[i] - math.log(dens)) < 1e-10
    one = orc.gmm_logpdf(x, logw[:, :1] + 3.0, mu[:, :1], ls[:, :1])          # weights are normalised inside
    np.testing.assert_allclose(one, orc.gaussian_logpdf_diag(x, mu[:, 0], 2 * ls[:, 0]), rtol=1e-12)


def test_gmm_sample_inverts_the_weight_cdf_and_follows_the_mixture():
    rng = np.random.default_rng(2)
    N = 100_000
    logw = np.log(np.array([0.2, 0.5, 0.3]))[None, :].repeat(N, 0)
    mu = np.array([-2.0, 0.0, 1.5])[None, :, None].repeat(N, 0)
    ls = np.log(np.array([0.5, 0.3, 1.0]))[None, :, None].repeat(N, 0)
    u, z = rng.random(N), rng.standard_normal((N, 1))
    x, comp = orc.gmm_sample(logw, mu, ls, u, z)
    np.testing.assert_array_equal(comp, np.digitize(u, [0.2, 0.7]))            # component = CDF inverse
    np.testing.assert_allclose(x[:, 0], mu[0, comp, 0] + np.exp(ls[0, comp, 0]) * z[:, 0], rtol=1e-12)
    cdf = lambda t: 0.2 * st.norm.cdf(t, -2.0, 0.5) + 0.5 * st.norm.cdf(t, 0.0, 0.3) + 0.3 * st.norm.cdf(t, 1.5, 1.0)
    assert st.kstest(x[:, 0], cdf).pvalue > 1e-3
    # u = 1 (beyond the rounded total) still picks the last component
    _, c1 = orc.gmm_sample(logw[:1], mu[:1], ls[:1], np.array([1.0]), z[:1])
    assert c1[0] == 2


def test_gmm_round_accepts_with_probability_one_minus_tv_and_resamples_the_positive_part():
    # 1-D mixtures, one position per sequence: P(accept) = E_q[min(1, p/q)] = 1 - TV(p, q); the resampled tokens
    # follow max(0, p - q)/Z (KS against the numerically integrated CDF); mean number of proposals = 1 / TV.
    rng = np.random.default_rng(3)
    N, cap = 100_000, 200
    qm = (np.log([0.6, 0.4]), np.array([[-1.0], [1.0]]), np.log([[0.7], [0.5]]))
    pm = (np.log([0.3, 0.7]), np.array([[-0.5], [1.4]]), np.log([[0.6], [0.6]]))
    rep = lambda m: tuple(np.broadcast_to(a, (N,) + np.shape(a)).copy() for a in m)
    q, p = rep(qm), rep(pm)
    out = orc.gmm_round(q, p, rng.random(N), rng.standard_normal((N, 1)), rng.random((N, 1)), rng.random((N, cap)),
                        rng.standard_normal((N, cap, 1)), rng.random((N, cap)), N, 1, cap)
    grid = np.linspace(-8, 8, 400_001)
    dens = lambda m: sum(np.exp(m[0][k]) * st.norm.pdf(grid, m[1][k][0], math.exp(m[2][k][0])) for k in range(2))
    pq = np.maximum(0.0, dens(pm) - dens(qm))
    tv = np.trapezoid(pq, grid)
    assert abs(out["n_accept"].mean() - (1.0 - tv)) < 0.006
    rej = out["flags"] & 1 == 1
    assert out["cap_hits"] == 0 and rej.sum() > 20_000
    cdf = np.concatenate([[0.0], np.cumsum(0.5 * (pq[1:] + pq[:-1]) * np.diff(grid))]) / tv
    assert st.kstest(out["x_new"][rej, 0], lambda t: np.interp(t, grid, cdf)).pvalue > 1e-3
    assert abs(out["n_prop"][rej].mean() - 1.0 / tv) < 0.03 / tv
    # power: plain draws from p fail the same test
    xp, _ = orc.gmm_sample(p[0], p[1], p[2], rng.random(N), rng.standard_normal((N, 1)))
    assert st.kstest(xp[:, 0], lambda t: np.interp(t, grid, cdf)).pvalue < 1e-6


def test_identical_mixtures_give_zero_ratio_and_accept_everything():
    rng = np.random.default_rng(4)
    B, gamma, K, C, cap = 5, 4, 3, 6, 4
    R = B * gamma
    m = _mix(rng, R, K, C)
    out = orc.gmm_round(m, m, rng.random(R), rng.standard_normal((R, C)), rng.random((B, gamma)), rng.random((B, cap)),
                        rng.standard_normal((B, cap, C)), rng.random((B, cap)), B, gamma, cap)
    assert np.all(out["logratio"] == 0.0) and np.all(out["n_accept"] == gamma) and np.all(out["flags"] == 0)
