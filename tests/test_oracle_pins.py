"""Pins of the float64 checker against what the paper and the mathematics fix.

None of these re-type the checker's formulas: each compares it with a closed
form, a library routine, a textbook identity, brute force, or a statistical
law, chosen so that a dropped term, a wrong sign/index or a transposed operand
in the checker breaks at least one of them.
"""
import itertools
import math

import numpy as np
import pytest
import scipy.stats as st
import torch

from oracle import csd_oracle as orc
from paper_2411_11925_b200 import inputs as gen


# ----------------------------------------------------------------- schedule
def test_schedule_unit_gaussian_data_gives_sqrt_alpha_posterior_mean():
    # Textbook: if x_0 ~ N(0,1) then every x_t ~ N(0,1), cov(x_t, x_{t-1}) = sqrt(alpha_t),
    # hence E[x_{t-1} | x_t] = sqrt(alpha_t) x_t.  The optimal eps-predictor plugged into the
    # DDPM mean must reproduce it; a wrong a_t or b_t cannot.
    beta = gen.beta_linear(50)
    s = orc.ddpm_schedule(beta)
    eps_fn = orc.make_gaussian_toy_head(0.0, 1.0, s["alphabar"])
    x = np.linspace(-3, 3, 11)[:, None]
    for t in (1, 2, 17, 50):
        mu = s["a"][t - 1] * x - s["b"][t - 1] * eps_fn(x, t)
        np.testing.assert_allclose(mu, math.sqrt(1.0 - beta[t - 1]) * x, rtol=0, atol=1e-13)


def test_schedule_point_mass_data_gives_ddpm_posterior_mean():
    # Ho et al. (DDPM) Eq. 7: for a known x_0 = m, the posterior mean of x_{t-1} given x_t is
    #   sqrt(ab_{t-1}) beta_t/(1-ab_t) m + sqrt(alpha_t)(1-ab_{t-1})/(1-ab_t) x_t.
    beta = gen.beta_linear(20)
    s = orc.ddpm_schedule(beta)
    ab = np.ones(21)
    for t in range(1, 21):
        ab[t] = ab[t - 1] * (1.0 - beta[t - 1])
    m = 0.7
    eps_fn = orc.make_gaussian_toy_head(m, 0.0, s["alphabar"])
    x = np.array([[-1.3], [0.2], [2.5]])
    for t in (2, 9, 20):
        mu = s["a"][t - 1] * x - s["b"][t - 1] * eps_fn(x, t)
        want = (math.sqrt(ab[t - 1]) * beta[t - 1] / (1 - ab[t]) * m
                + math.sqrt(1 - beta[t - 1]) * (1 - ab[t - 1]) / (1 - ab[t]) * x)
        np.testing.assert_allclose(mu, want, rtol=0, atol=1e-13)


@pytest.mark.parametrize("eta", [0.3, 1.0])
def test_ddim_schedule_preserves_gaussian_marginals(eta):
    # Defining property of DDIM: given the true x_0, for every sigma the reverse step maps the marginal of x_t
    # onto that of x_prev.  Point-mass data x_0 = m (the predictor then returns the true noise):
    # x_t ~ N(sqrt(ab) m, 1 - ab), the step is affine x_prev = A x_t + D + sigma eps, so mean and variance can
    # be pushed through by hand.
    N, m, s_ = 200, 0.7, 0.0
    beta = gen.beta_linear(N)
    steps = np.arange(10, N + 1, 10)
    sch = orc.ddim_schedule(beta, steps, eta)
    eps_fn = orc.make_gaussian_toy_head(m, s_, sch["alphabar"])
    ab = sch["alphabar"]
    for k in range(len(steps), 1, -1):           # steps with a proper predecessor marginal (ab_prev < 1)
        x = np.array([[0.0], [1.0]])
        mu = sch["a"][k - 1] * x - sch["b"][k - 1] * eps_fn(x, k)
        A, D = mu[1, 0] - mu[0, 0], mu[0, 0]
        mean_t, var_t = math.sqrt(ab[k - 1]) * m, ab[k - 1] * s_ ** 2 + 1 - ab[k - 1]
        mean_p, var_p = math.sqrt(ab[k - 2]) * m, ab[k - 2] * s_ ** 2 + 1 - ab[k - 2]
        assert abs(A * mean_t + D - mean_p) < 1e-12
        assert abs(A * A * var_t + sch["sigma"][k - 1] ** 2 - var_p) < 1e-12


def test_ddim_with_eta_one_on_the_full_ladder_is_the_ddpm_posterior():
    # Song et al.: eta = 1 recovers DDPM: same mean coefficients as the eps-parameterised DDPM mean and the posterior
    # variance beta~_t = (1 - ab_{t-1}) / (1 - ab_t) beta_t (Ho et al., Eq. 7).
    T = 30
    beta = gen.beta_linear(T)
    dd, dp = orc.ddim_schedule(beta, np.arange(1, T + 1), 1.0), orc.ddpm_schedule(beta)
    ab = np.cumprod(1 - beta)
    np.testing.assert_allclose(dd["a"], dp["a"], rtol=1e-12)
    np.testing.assert_allclose(dd["b"][1:], dp["b"][1:], rtol=1e-10)
    np.testing.assert_allclose(dd["sigma"][1:] ** 2, (1 - ab[:-1]) / (1 - ab[1:]) * beta[1:], rtol=1e-12)
    # last step: the mean is the predicted x_0 (for point-mass data it is the data point itself)
    eps_fn = orc.make_gaussian_toy_head(0.4, 0.0, dd["alphabar"])
    x = np.array([[-1.0], [2.5]])
    np.testing.assert_allclose(dd["a"][0] * x - dd["b"][0] * eps_fn(x, 1), 0.4, atol=1e-12)
    assert abs(dd["sigma"][0] - math.sqrt(1 - ab[0])) < 1e-15


def test_temperature_scales_sigma_only():
    beta = gen.beta_linear(10)
    s1, s2 = orc.ddpm_schedule(beta, 1.0), orc.ddpm_schedule(beta, 0.8)
    np.testing.assert_allclose(s2["sigma"], 0.8 * np.sqrt(beta), rtol=1e-15)
    np.testing.assert_array_equal(s1["a"], s2["a"])
    np.testing.assert_array_equal(s1["b"], s2["b"])


# ------------------------------------------------------- head building blocks
def test_silu_and_layer_norm_match_library_routines():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 37)) * 3.0
    xt = torch.from_numpy(x)
    np.testing.assert_allclose(orc.silu(x), torch.nn.functional.silu(xt).numpy(), atol=1e-14)
    np.testing.assert_allclose(orc.layer_norm(x),
                               torch.nn.functional.layer_norm(xt, (37,), eps=1e-6).numpy(),
                               atol=1e-12)


def _torch_linear(W, b, x):
    return torch.nn.functional.linear(torch.from_numpy(np.asarray(x, dtype=np.float64)),
                                      torch.from_numpy(W.astype(np.float64)),
                                      torch.from_numpy(b.astype(np.float64))).numpy()


def test_timestep_embedding_matches_library_mlp():
    spec = gen.HeadSpec(L=1, W=24, Dz=10, C=3, F=8)
    w = gen.make_head_weights(spec, np.random.default_rng(1))
    tf = gen.timestep_features(6, 8)
    for t in (1, 6):
        hid = torch.nn.functional.silu(torch.from_numpy(_torch_linear(w["Wt1"], w["bt1"], tf[t - 1])))
        want = _torch_linear(w["Wt2"], w["bt2"], hid.numpy())
        np.testing.assert_allclose(orc.timestep_embedding(w, tf[t - 1]), want, atol=1e-13)


def test_head_with_neutral_modulation_reduces_to_plain_residual_mlp():
    # With AdaLN weights/biases zero except gate bias 1: shift=scale=0, gate=1, so every block is
    # h + W2 SiLU(W1 LN(h) + b1) + b2 and the output is Wout LN(h) + bout: all library routines.
    # Non-square shapes (C=3, W=24, Dz=10, F=8) make any transposed operand a shape error.
    spec = gen.HeadSpec(L=2, W=24, Dz=10, C=3, F=8)
    w = gen.make_head_weights(spec, np.random.default_rng(2))
    w["Wada"][:] = 0; w["bada"][:] = 0; w["bada"][:, 2 * 24:] = 1.0
    w["Wfada"][:] = 0; w["bfada"][:] = 0
    rng = np.random.default_rng(3)
    x, z = rng.standard_normal((4, 3)), rng.standard_normal((4, 10))
    tf = gen.timestep_features(4, 8)
    ln = lambda a: torch.nn.functional.layer_norm(torch.from_numpy(a), (24,), eps=1e-6).numpy()
    h = _torch_linear(w["Win"], w["bin"], x)
    for k in range(2):
        a = torch.nn.functional.silu(torch.from_numpy(_torch_linear(w["W1"][k], w["b1"][k], ln(h)))).numpy()
        h = h + _torch_linear(w["W2"][k], w["b2"][k], a)
    want = _torch_linear(w["Wout"], w["bout"], ln(h))
    np.testing.assert_allclose(orc.head_eps(w, x, tf[2], z), want, atol=1e-12)


def test_head_modulation_terms_each_matter_and_enter_as_specified():
    # One block, W=4: u = LN(h)(1+scale)+shift, h' = h + gate*MLP(u).  Making only the
    # modulation *biases* non-zero gives constant shift/scale/gate, which library routines
    # reproduce; checks the (shift | scale | gate) split order and the (shift | scale) order
    # of the final layer.
    W = 4
    spec = gen.HeadSpec(L=1, W=W, Dz=5, C=2, F=6)
    w = gen.make_head_weights(spec, np.random.default_rng(4))
    w["Wada"][:] = 0; w["Wfada"][:] = 0
    sh, sc, ga = 0.3, -0.2, 0.7
    w["bada"][0, :W], w["bada"][0, W:2 * W], w["bada"][0, 2 * W:] = sh, sc, ga
    fsh, fsc = -0.4, 0.5
    w["bfada"][:W], w["bfada"][W:] = fsh, fsc
    rng = np.random.default_rng(5)
    x, z = rng.standard_normal((3, 2)), rng.standard_normal((3, 5))
    tf = gen.timestep_features(3, 6)
    ln = lambda a: torch.nn.functional.layer_norm(torch.from_numpy(a), (W,), eps=1e-6).numpy()
    h = _torch_linear(w["Win"], w["bin"], x)
    u = ln(h) * (1 + np.float32(sc).astype(np.float64)) + np.float64(np.float32(sh))
    a = torch.nn.functional.silu(torch.from_numpy(_torch_linear(w["W1"][0], w["b1"][0], u))).numpy()
    h = h + np.float64(np.float32(ga)) * _torch_linear(w["W2"][0], w["b2"][0], a)
    uf = ln(h) * (1 + np.float64(np.float32(fsc))) + np.float64(np.float32(fsh))
    want = _torch_linear(w["Wout"], w["bout"], uf)
    np.testing.assert_allclose(orc.head_eps(w, x, tf[0], z), want, atol=1e-12)


def test_head_condition_path_is_silu_of_cz_plus_te_through_adaln():
    # s = SiLU(Wz z + bz + te_t) feeds the modulation: compare the scale/shift/gate the head
    # derives (traced) against library linear algebra on s; the z and t dependence must be live.
    spec = gen.HeadSpec(L=1, W=8, Dz=5, C=2, F=6)
    w = gen.make_head_weights(spec, np.random.default_rng(6))
    rng = np.random.default_rng(7)
    x, z = rng.standard_normal((3, 2)), rng.standard_normal((3, 5))
    tf = gen.timestep_features(3, 6)
    tr = {}
    e1 = orc.head_eps(w, x, tf[0], z, trace=tr)
    te = orc.timestep_embedding(w, tf[0])
    s = torch.nn.functional.silu(torch.from_numpy(_torch_linear(w["Wz"], w["bz"], z) + te)).numpy()
    np.testing.assert_allclose(tr["s"], s, atol=1e-13)
    assert np.max(np.abs(orc.head_eps(w, x, tf[2], z) - e1)) > 1e-6       # t matters
    assert np.max(np.abs(orc.head_eps(w, x, tf[0], z[::-1].copy()) - e1)) > 1e-6  # z matters


def test_cfg_combination_is_linear_extrapolation():
    spec = gen.HeadSpec(L=1, W=16, Dz=6, C=4, F=8)
    w = gen.make_head_weights(spec, np.random.default_rng(8))
    rng = np.random.default_rng(9)
    R = 5
    x, z = rng.standard_normal((R, 4)), rng.standard_normal((2 * R, 6))
    tf = gen.timestep_features(3, 8)
    e_c = orc.head_eps(w, x, tf[1], z[:R]); e_u = orc.head_eps(w, x, tf[1], z[R:])
    for scale in (0.0, 1.0, 3.0):
        got = orc.make_mlp_head(w, z, tf, True, scale)(x, 2)
        np.testing.assert_allclose(got, (1 - scale) * e_u + scale * e_c, atol=1e-13)


# ---------------------------------------------------- trajectories & Theorem 1
def _toy_pair(T=12, C=3, tau_q=1.0, tau_p=1.0):
    beta = gen.beta_linear(T)
    sq, sp = orc.ddpm_schedule(beta, tau_q), orc.ddpm_schedule(beta, tau_p)
    eq = orc.make_gaussian_toy_head(0.3, 0.8, sq["alphabar"])
    ep = orc.make_gaussian_toy_head(-0.1, 1.1, sp["alphabar"])
    return beta, sq, sp, eq, ep


def test_theorem1_pathwise_difference_equals_mean_difference():
    # Theorem 1 (aligned case): x^q_{t-1} - x^p_{t-1} = (mu^q_t - mu^p_t) + (sigma_q - sigma_p) eps_t.
    _, sq, sp, eq, ep = _toy_pair(tau_p=0.9)
    rng = np.random.default_rng(10)
    x_T, noise = rng.standard_normal((7, 3)), rng.standard_normal((12, 7, 3))
    dq, dp = orc.run_pair(eq, ep, sq, sp, x_T, noise, keep=True)
    for j in range(11):                      # steps t = T..2
        t = 12 - j
        lhs = dq["xs"][j + 1] - dp["xs"][j + 1]
        rhs = dq["mus"][j] - dp["mus"][j] + (sq["sigma"][t - 1] - sp["sigma"][t - 1]) * noise[t - 1]
        np.testing.assert_allclose(lhs, rhs, atol=1e-13)


def test_theorem1_alignment_reduces_expected_distance_by_2_tr_sqrt():
    # Monte Carlo over the noise of the first step, same x_T: E_unaligned - E_aligned
    # = 2 tr sqrt(Sigma_q Sigma_p) = 2 C sigma_q sigma_p (boxed identities of the proof).
    T, C, N = 2, 4, 400_000
    beta = gen.beta_linear(T, 0.05, 0.2)
    sq, sp = orc.ddpm_schedule(beta, 1.0), orc.ddpm_schedule(beta, 0.7)
    eq = orc.make_gaussian_toy_head(0.3, 0.8, sq["alphabar"])
    ep = orc.make_gaussian_toy_head(-0.1, 1.1, sp["alphabar"])
    rng = np.random.default_rng(11)
    x_T = np.tile(rng.standard_normal((1, C)), (N, 1))
    noise, noise2 = rng.standard_normal((T, N, C)), rng.standard_normal((T, N, C))
    dq, dp = orc.run_pair(eq, ep, sq, sp, x_T, noise)
    _, dp_un = orc.run_pair(eq, ep, sq, sp, x_T, noise, noise_p=noise2)
    d_al = np.mean(np.sum((dq["x1"] - dp["x1"]) ** 2, axis=1))
    d_un = np.mean(np.sum((dq["x1"] - dp_un["x1"]) ** 2, axis=1))
    want = 2 * C * sq["sigma"][1] * sp["sigma"][1]
    assert abs((d_un - d_al) - want) < 0.02 * want
    # and the aligned value itself: ||mu_q-mu_p||^2 + C (sigma_p - sigma_q)^2
    mu_q = sq["a"][1] * x_T[0] - sq["b"][1] * eq(x_T[:1], 2)[0]
    mu_p = sp["a"][1] * x_T[0] - sp["b"][1] * ep(x_T[:1], 2)[0]
    al = np.sum((mu_q - mu_p) ** 2) + C * (sp["sigma"][1] - sq["sigma"][1]) ** 2
    assert abs(d_al - al) < 0.02 * al + 1e-4


def test_target_never_samples_x0_and_draft_adds_noise_at_last_step():
    _, sq, sp, eq, ep = _toy_pair()
    rng = np.random.default_rng(12)
    x_T, noise = rng.standard_normal((3, 3)), rng.standard_normal((12, 3, 3))
    dq, dp = orc.run_pair(eq, ep, sq, sp, x_T, noise)
    assert dp["x0"] is None
    np.testing.assert_allclose(dq["x0"], dq["mu1"] + sq["sigma"][0] * noise[0], atol=1e-15)


# ---------------------------------------------------------------- log-ratio
def test_long_product_equals_sigma_times_final_step_ratio():
    # Eq. 4 (product over all T steps) == Eq. 8 (Sigma * final-step ratio) under alignment,
    # also with sigma_q != sigma_p so that Sigma (Eq. 7) is not 1.
    for tau_p in (1.0, 0.85):
        _, sq, sp, eq, ep = _toy_pair(tau_p=tau_p)
        rng = np.random.default_rng(13)
        x_T, noise = rng.standard_normal((9, 3)), rng.standard_normal((12, 9, 3))
        dq, dp = orc.run_pair(eq, ep, sq, sp, x_T, noise, keep=True)
        ls = orc.log_sigma_term(sq["sigma"], sp["sigma"], 3)
        closed = orc.log_ratio_closed(dq["x0"], dq["mu1"], dp["mu1"], sq["sigma"][0], sp["sigma"][0], ls)
        np.testing.assert_allclose(orc.log_ratio_long(dq, dp, sq, sp), closed, atol=1e-9)
        if tau_p == 1.0:
            assert ls == 0.0
        else:   # Sigma = prod_{t>=2} (sigma_q/sigma_p)^C = tau_p^{-C (T-1)}
            assert abs(ls - (-3 * 11 * math.log(tau_p))) < 1e-10


def test_unaligned_long_product_differs_from_closed_form():
    # Without alignment the per-step exponentials do not cancel: guards against a long form
    # that ignores the trajectories.
    _, sq, sp, eq, ep = _toy_pair()
    rng = np.random.default_rng(14)
    x_T, noise, noise2 = rng.standard_normal((4, 3)), rng.standard_normal((12, 4, 3)), rng.standard_normal((12, 4, 3))
    dq, dp = orc.run_pair(eq, ep, sq, sp, x_T, noise, noise_p=noise2, keep=True)
    closed = orc.log_ratio_closed(dq["x0"], dq["mu1"], dp["mu1"], sq["sigma"][0], sp["sigma"][0], 0.0)
    assert np.min(np.abs(orc.log_ratio_long(dq, dp, sq, sp) - closed)) > 1e-3


def test_gaussian_logpdf_matches_scipy():
    rng = np.random.default_rng(15)
    x, mu = rng.standard_normal((6, 5)), rng.standard_normal((6, 5))
    want = st.norm.logpdf(x, loc=mu, scale=0.37).sum(axis=1)
    np.testing.assert_allclose(orc.gaussian_logpdf_iso(x, mu, 0.37), want, atol=1e-12)


def test_identical_heads_give_exactly_zero_logratio_and_accept_everything():
    wl = gen.WORKLOADS["tiny_fp32"]
    inp = gen.make_round_inputs(wl)
    inp.w_q, inp.z_q = inp.w_p, inp.z_p
    out = orc.round_from_inputs(inp)
    assert np.all(out["logratio"] == 0.0)
    assert np.all(out["n_accept"] == wl.gamma)
    assert np.all(out["flags"] == 0) and np.all(out["n_prop"] == 0)


def test_toy_gaussian_logratio_matches_independent_affine_composition():
    # 1-D Gaussian toy heads make every step affine: x_{t-1} = A_t x_t + D_t + sigma_t eps_t.
    # Solve the whole trajectory as ONE bidiagonal linear system (no stepping), then evaluate
    # the final-step ratio with scipy's normal density.
    T = 25
    beta = gen.beta_linear(T)
    tau_q, tau_p = 1.0, 0.9
    sq, sp = orc.ddpm_schedule(beta, tau_q), orc.ddpm_schedule(beta, tau_p)
    heads = {"q": (0.4, 0.6), "p": (-0.2, 0.9)}
    eq = orc.make_gaussian_toy_head(*heads["q"], sq["alphabar"])
    ep = orc.make_gaussian_toy_head(*heads["p"], sp["alphabar"])
    rng = np.random.default_rng(16)
    N = 6
    x_T, noise = rng.standard_normal((N, 1)), rng.standard_normal((T, N, 1))
    dq, dp = orc.run_pair(eq, ep, sq, sp, x_T, noise)
    ls = orc.log_sigma_term(sq["sigma"], sp["sigma"], 1)
    got = orc.log_ratio_closed(dq["x0"], dq["mu1"], dp["mu1"], sq["sigma"][0], sp["sigma"][0], ls)

    ab = np.cumprod(1 - beta)

    def coeffs(m, s, t):
        k = math.sqrt(1 - ab[t - 1]) / (ab[t - 1] * s * s + 1 - ab[t - 1])
        bt = beta[t - 1] / (math.sqrt(1 - beta[t - 1]) * math.sqrt(1 - ab[t - 1]))
        return 1 / math.sqrt(1 - beta[t - 1]) - bt * k, bt * k * math.sqrt(ab[t - 1]) * m

    def x1_and_mu1(m, s, tau, xT, nz):
        # unknowns y = (x_{T-1}, ..., x_1): x_{t-1} - A_t x_t = D_t + sigma_t eps_t
        M = np.eye(T - 1); rhs = np.zeros(T - 1)
        for i, t in enumerate(range(T, 1, -1)):
            A, D = coeffs(m, s, t)
            rhs[i] = D + tau * math.sqrt(beta[t - 1]) * nz[t - 1]
            if i == 0:
                rhs[i] += A * xT
            else:
                M[i, i - 1] = -A
        x1 = np.linalg.solve(M, rhs)[-1]
        A1, D1 = coeffs(m, s, 1)
        return x1, A1 * x1 + D1

    for r in range(N):
        _, mu_q = x1_and_mu1(*heads["q"], tau_q, x_T[r, 0], noise[:, r, 0])
        _, mu_p = x1_and_mu1(*heads["p"], tau_p, x_T[r, 0], noise[:, r, 0])
        s1q, s1p = tau_q * math.sqrt(beta[0]), tau_p * math.sqrt(beta[0])
        x0 = mu_q + s1q * noise[0, r, 0]
        want = ((T - 1) * math.log(tau_q / tau_p)
                + st.norm.logpdf(x0, mu_p, s1p) - st.norm.logpdf(x0, mu_q, s1q))
        assert abs(got[r] - want) < 1e-8 * max(1.0, abs(want))


# ------------------------------------------------- single-path exact ratio (Eq. 2)
def test_single_path_ratio_with_one_step_is_the_final_step_ratio():
    # T = 1: both trajectories consist of x_T = x_1 only, so Eq. 2 and Eq. 8 coincide (Sigma = 1).
    beta = gen.beta_linear(1, 0.02, 0.02)
    sq, sp = orc.ddpm_schedule(beta, 1.0), orc.ddpm_schedule(beta, 0.8)
    eq = orc.make_gaussian_toy_head(0.3, 0.8, sq["alphabar"])
    ep = orc.make_gaussian_toy_head(-0.1, 1.1, sp["alphabar"])
    rng = np.random.default_rng(40)
    x_T, noise = rng.standard_normal((5, 3)), rng.standard_normal((1, 5, 3))
    dq, dp = orc.run_pair(eq, ep, sq, sp, x_T, noise, keep=True)
    closed = orc.log_ratio_closed(dq["x0"], dq["mu1"], dp["mu1"], sq["sigma"][0], sp["sigma"][0], 0.0)
    np.testing.assert_allclose(orc.log_ratio_single_path(ep, sq, sp, dq), closed, atol=1e-12)


def test_single_path_ratio_of_identical_heads_is_exactly_zero():
    wl = gen.WORKLOADS["tiny_fp32"]
    inp = gen.make_round_inputs(wl)
    inp.w_q, inp.z_q = inp.w_p, inp.z_p
    out = orc.single_path_from_inputs(inp)
    assert np.all(out["logratio"] == 0.0) and np.all(out["n_accept"] == wl.gamma)
    assert out["traj_x"].shape == (wl.T + 1, wl.R, 16) and out["traj_mu"].shape == (wl.T, wl.R, 16)


def _toy_path_gaussian(m, s, tau, beta, xT):
    # 1-D Gaussian toy head: x_{t-1} = A_t x_t + D_t + sigma_t eps_t.  The path y = (x_{T-1}, ..., x_0) given
    # x_T solves M y = d + S eps, hence y ~ N(M^-1 d, M^-1 S S^T M^-T).
    T = len(beta)
    ab = np.cumprod(1 - beta)
    M, d, S = np.eye(T), np.zeros(T), np.zeros((T, T))
    for i, t in enumerate(range(T, 0, -1)):
        k = math.sqrt(1 - ab[t - 1]) / (ab[t - 1] * s * s + 1 - ab[t - 1])
        bt = beta[t - 1] / (math.sqrt(1 - beta[t - 1]) * math.sqrt(1 - ab[t - 1]))
        A, D = 1 / math.sqrt(1 - beta[t - 1]) - bt * k, bt * k * math.sqrt(ab[t - 1]) * m
        d[i] = D + (A * xT if i == 0 else 0.0)
        if i > 0:
            M[i, i - 1] = -A
        S[i, i] = tau * math.sqrt(beta[t - 1])
    Minv = np.linalg.inv(M)
    return Minv @ d, Minv @ S @ S.T @ Minv.T


def test_single_path_ratio_matches_multivariate_normal_path_densities():
    # With toy heads the whole path given x_T is jointly Gaussian under either model, so Eq. 2 is the difference
    # of two multivariate-normal log-densities (scipy), evaluated at the draft's path: no stepping, no per-step terms.
    T = 8
    beta = gen.beta_linear(T, 0.01, 0.2)
    tau_q, tau_p = 1.0, 0.9
    sq, sp = orc.ddpm_schedule(beta, tau_q), orc.ddpm_schedule(beta, tau_p)
    eq = orc.make_gaussian_toy_head(0.4, 0.6, sq["alphabar"])
    ep = orc.make_gaussian_toy_head(-0.2, 0.9, sp["alphabar"])
    rng = np.random.default_rng(41)
    N = 5
    x_T, noise = rng.standard_normal((N, 1)), rng.standard_normal((T, N, 1))
    dq = orc.denoise(eq, sq, x_T, noise, sample_last=True, keep=True)
    got = orc.log_ratio_single_path(ep, sq, sp, dq)
    for r in range(N):
        y = np.array([dq["xs"][j + 1][r, 0] for j in range(T)])
        mq, cq = _toy_path_gaussian(0.4, 0.6, tau_q, beta, x_T[r, 0])
        mp, cp = _toy_path_gaussian(-0.2, 0.9, tau_p, beta, x_T[r, 0])
        want = st.multivariate_normal(mp, cp).logpdf(y) - st.multivariate_normal(mq, cq).logpdf(y)
        assert abs(got[r] - want) < 1e-8 * max(1.0, abs(want))


def test_unaligned_long_product_matches_multivariate_normal_path_densities():
    # Ablation without trajectory alignment (the target draws its own noise): p(Y_p)/q(Y_q) of Eq. 4 is the joint
    # density of the target's path (ending in the draft's x_0) under p over that of the draft's path under q; with toy
    # heads both joints are multivariate normal (scipy), no per-step terms involved.
    T = 7
    beta = gen.beta_linear(T, 0.01, 0.2)
    tau_q, tau_p = 1.0, 0.9
    sq, sp = orc.ddpm_schedule(beta, tau_q), orc.ddpm_schedule(beta, tau_p)
    eq = orc.make_gaussian_toy_head(0.4, 0.6, sq["alphabar"])
    ep = orc.make_gaussian_toy_head(-0.2, 0.9, sp["alphabar"])
    rng = np.random.default_rng(43)
    N = 5
    x_T = rng.standard_normal((N, 1))
    noise, noise_p = rng.standard_normal((T, N, 1)), rng.standard_normal((T, N, 1))
    dq, dp = orc.run_pair(eq, ep, sq, sp, x_T, noise, noise_p=noise_p, keep=True)
    got = orc.log_ratio_long(dq, dp, sq, sp)
    for r in range(N):
        yq = np.array([dq["xs"][j + 1][r, 0] for j in range(T)])
        yp = np.array([dp["xs"][j + 1][r, 0] for j in range(T - 1)] + [dq["x0"][r, 0]])
        mq, cq = _toy_path_gaussian(0.4, 0.6, tau_q, beta, x_T[r, 0])
        mp, cp = _toy_path_gaussian(-0.2, 0.9, tau_p, beta, x_T[r, 0])
        want = st.multivariate_normal(mp, cp).logpdf(yp) - st.multivariate_normal(mq, cq).logpdf(yq)
        assert abs(got[r] - want) < 1e-8 * max(1.0, abs(want))


def test_single_path_ratio_has_unit_expectation_under_the_draft():
    # E_{Y ~ q}[p(Y)/q(Y)] = 1 (importance-weight identity stated with the bias analysis of the surrogate ratio);
    # a dropped step, a wrong sign or a wrong variance in Eq. 2 breaks it.
    T, N = 3, 400_000
    beta = gen.beta_linear(T, 0.05, 0.2)
    sq, sp = orc.ddpm_schedule(beta, 1.0), orc.ddpm_schedule(beta, 0.95)
    eq = orc.make_gaussian_toy_head(0.1, 0.9, sq["alphabar"])
    ep = orc.make_gaussian_toy_head(0.0, 1.0, sp["alphabar"])
    rng = np.random.default_rng(42)
    x_T = np.tile(rng.standard_normal((1, 1)), (N, 1))
    noise = rng.standard_normal((T, N, 1))
    dq = orc.denoise(eq, sq, x_T, noise, sample_last=True, keep=True)
    w = np.exp(orc.log_ratio_single_path(ep, sq, sp, dq))
    se = w.std() / math.sqrt(N)
    assert abs(w.mean() - 1.0) < 5 * se + 1e-3, (w.mean(), se)
    assert w.std() > 0.05          # not vacuous: the two models differ


def test_bonus_token_is_a_target_sample_exactly_where_everything_was_accepted():
    # The all-accepted branch of Alg. 1: on Gaussian data with point mass m the target's samples end within a few
    # sigma_1 of m (its reverse process contracts onto the data), and only sequences with n = gamma receive one.
    T, B, gamma = 40, 6, 4
    sp = orc.ddpm_schedule(gen.beta_linear(T))
    ep = orc.make_gaussian_toy_head(0.25, 0.0, sp["alphabar"])
    rng = np.random.default_rng(50)
    x_T, noise = rng.standard_normal((B, 2)), rng.standard_normal((T, B, 2))
    n = np.array([4, 0, 3, 4, 2, 4])
    out = orc.bonus_token(ep, sp, x_T, noise, n, gamma)
    np.testing.assert_array_equal(out["taken"], [True, False, False, True, False, True])
    assert np.all(out["x_bonus"][~out["taken"]] == 0.0)
    assert np.all(np.abs(out["x_bonus"][out["taken"]] - 0.25) < 6 * sp["sigma"][0])
    # and it is the last state of the plain reverse process with noise at every step
    d = orc.denoise(ep, sp, x_T, noise, sample_last=True)
    np.testing.assert_array_equal(out["x_bonus"][out["taken"]], d["x0"][out["taken"]])
    np.testing.assert_allclose(d["x0"], d["mu1"] + sp["sigma"][0] * noise[0], atol=1e-15)


# --------------------------------------------------------------- accept scan
@pytest.mark.parametrize("gamma", [1, 3, 8])
def test_accept_prefix_brute_force_all_masks(gamma):
    masks = list(itertools.product([0, 1], repeat=gamma))
    logr = np.full((len(masks), gamma), math.log(0.5))
    u = np.array([[0.25 if a else 0.75 for a in m] for m in masks])
    n, acc = orc.accept_prefix(logr, u)
    for b, m in enumerate(masks):
        s = "".join(map(str, m))
        want = s.find("0") if "0" in s else gamma          # first reject, else gamma
        assert n[b] == want
        assert tuple(acc[b].astype(int)) == m


def test_accept_rule_boundary_and_ratio_above_one():
    # accept iff r <= p/q: equality accepts; ratio > 1 always accepts (Alg. 1, Fig. 3 caption)
    logr = np.array([[math.log(0.5), math.log(0.5), 2.0, -1e9]])
    u = np.array([[0.5, np.nextafter(0.5, 1.0), 0.999999, 1e-30]])
    n, acc = orc.accept_prefix(logr, u)
    assert list(acc[0]) == [True, False, True, False] and n[0] == 1


def test_accept_rate_is_expected_min_one_ratio():
    rng = np.random.default_rng(17)
    logr = np.full((200_000, 1), math.log(0.3))
    n, _ = orc.accept_prefix(logr, rng.random((200_000, 1)))
    assert abs(n.mean() - 0.3) < 0.005


# ----------------------------------------------------------------- resampler
def _resample_draws(mu_p, mu_q, s_p, s_q, log_sigma, N, cap, seed):
    rng = np.random.default_rng(seed)
    xi, v = rng.standard_normal((N, cap, 1)), rng.random((N, cap))
    out = orc.resample(np.zeros(N, dtype=np.int32), np.full((N, 1), mu_p), np.full((N, 1), mu_q),
                       s_p, s_q, log_sigma, xi, v, gamma=1, cap=cap)
    return out


def _modified_cdf(mu_p, mu_q, s_p, s_q, log_sigma):
    grid = np.linspace(min(mu_p, mu_q) - 12 * max(s_p, s_q), max(mu_p, mu_q) + 12 * max(s_p, s_q), 400_001)
    dens = np.maximum(0.0, math.exp(log_sigma) * st.norm.pdf(grid, mu_p, s_p) - st.norm.pdf(grid, mu_q, s_q))
    cdf = np.concatenate([[0.0], np.cumsum(0.5 * (dens[1:] + dens[:-1]) * np.diff(grid))])
    Z = cdf[-1]
    return (lambda x: np.interp(x, grid, cdf / Z)), Z


@pytest.mark.parametrize("mu_p,mu_q,s_p,s_q,log_sigma", [
    (0.0, 0.8, 1.0, 1.0, 0.0),          # equal variances, Sigma = 1
    (0.2, -0.1, 0.7, 1.0, 0.0),         # different variances
    (0.0, 0.5, 1.0, 0.9, 0.35),         # Sigma != 1
])
def test_resampled_tokens_follow_normalised_positive_part(mu_p, mu_q, s_p, s_q, log_sigma):
    N = 100_000
    out = _resample_draws(mu_p, mu_q, s_p, s_q, log_sigma, N, cap=400, seed=18)
    assert out["cap_hits"] == 0 and np.all(out["flags"] == 1)
    cdf, Z = _modified_cdf(mu_p, mu_q, s_p, s_q, log_sigma)
    res = st.kstest(out["x_new"][:, 0], cdf)
    assert res.pvalue > 1e-3, res
    # loop acceptance probability = Z / Sigma  =>  mean #proposals = Sigma / Z (geometric law)
    assert abs(out["n_prop"].mean() - math.exp(log_sigma) / Z) < 0.03 * math.exp(log_sigma) / Z
    # a sample from the plain target p would fail the same test: the test has power
    assert st.kstest(np.random.default_rng(1).normal(mu_p, s_p, N), cdf).pvalue < 1e-6


def test_resample_acceptance_rate_is_total_variation_distance():
    # Sigma = 1 and equal sigma: P(accept one proposal) = TV(p, q) = 2 Phi(|dmu| / (2 sigma)) - 1,
    # in any dimension (here C = 16 through the general code path).
    C, N, cap = 16, 20_000, 1
    rng = np.random.default_rng(19)
    mu_p = np.tile(rng.standard_normal((1, C)), (N, 1)); d = 0.9 * rng.standard_normal(C)
    mu_q = mu_p + d
    xi, v = rng.standard_normal((N, cap, C)), rng.random((N, cap))
    out = orc.resample(np.zeros(N, dtype=np.int32), mu_p, mu_q, 1.3, 1.3, 0.0, xi, v, gamma=1, cap=cap)
    acc_rate = np.mean((out["flags"] & 2) == 0)
    tv = 2 * st.norm.cdf(np.linalg.norm(d) / (2 * 1.3)) - 1
    assert abs(acc_rate - tv) < 4 * math.sqrt(tv * (1 - tv) / N)


def test_resample_indexing_cap_and_untouched_rows():
    gamma, cap, C = 3, 2, 2
    mu_p = np.arange(2 * gamma * C, dtype=float).reshape(2 * gamma, C)
    mu_q = mu_p + 100.0                       # q negligible at proposals => alpha_s = 1
    xi = np.ones((2, cap, C)); v = np.full((2, cap), 0.5)
    out = orc.resample(np.array([1, gamma]), mu_p, mu_q, 0.5, 0.5, 0.0, xi, v, gamma, cap)
    np.testing.assert_allclose(out["x_new"][0], mu_p[0 * gamma + 1] + 0.5)   # row b*gamma + n
    assert out["n_prop"][0] == 1 and out["flags"][0] == 1
    assert out["n_prop"][1] == 0 and out["flags"][1] == 0                    # n = gamma: untouched
    # identical p and q: alpha_s = 0 always -> cap hit, last proposal returned, flagged
    xi2 = np.stack([np.ones((cap, C)), 2 * np.ones((cap, C))]); xi2[:, 1] *= 3
    out = orc.resample(np.array([0, 0]), mu_p, mu_p, 0.5, 0.5, 0.0, xi2, v, gamma, cap)
    assert list(out["flags"]) == [3, 3] and out["cap_hits"] == 2 and list(out["n_prop"]) == [cap, cap]
    np.testing.assert_allclose(out["x_new"][1], mu_p[gamma] + 0.5 * xi2[1, cap - 1])


def test_resample_threshold_matches_direct_density_formula():
    # Cor. 1 in probability space (no logs) on a benign case.
    rng = np.random.default_rng(20)
    mu_p, mu_q = rng.standard_normal((1, 3)), rng.standard_normal((1, 3))
    xi = rng.standard_normal((1, 1, 3))
    out = orc.resample(np.array([0]), mu_p, mu_q, 0.8, 1.1, 0.2, xi, np.array([[2.0]]), 1, 1)
    xp = mu_p[0] + 0.8 * xi[0, 0]
    p = math.exp(0.2) * np.prod(st.norm.pdf(xp, mu_p[0], 0.8)); q = np.prod(st.norm.pdf(xp, mu_q[0], 1.1))
    assert abs(out["alpha_first"][0] - max(0.0, p - q) / p) < 1e-12


# ------------------------------------------------------------ whole round
def test_round_is_deterministic_and_matches_stored_reference():
    import json, os
    wl = gen.WORKLOADS["tiny_fp32"]
    out = orc.round_from_inputs(gen.make_round_inputs(wl))
    out2 = orc.round_from_inputs(gen.make_round_inputs(wl))
    np.testing.assert_array_equal(out["x0"], out2["x0"])
    path = os.path.join(os.path.dirname(__file__), "golden", "tiny_fp32_round.json")
    ref = json.load(open(path))
    np.testing.assert_allclose(out["x0"], np.array(ref["x0"]), atol=1e-12)
    np.testing.assert_allclose(out["logratio"], np.array(ref["logratio"]), atol=1e-9)
    assert list(out["n_accept"]) == ref["n_accept"]
