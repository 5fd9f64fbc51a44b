"""GPU parity of a whole round when both heads are sampled with DDIM instead of DDPM (the sampler enters only through
the transition coefficients a, b, sigma and the feature rows of the visited timesteps)."""
import numpy as np
import pytest

from oracle import csd_oracle as orc
from paper_2411_11925_b200 import inputs as gen

from _parity import compare_round

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("op,kw,eta_q,eta_p", [
    ("f32", dict(B=4, gamma=4, T=10), 1.0, 1.0),
    ("f32", dict(B=4, gamma=5, T=8, cfg=True, cfg_scale=2.0), 0.7, 0.5),      # sigma_q != sigma_p: Sigma of Eq. 7 != 1
    ("f16", dict(B=9, gamma=8, T=8, bf16=True, cfg=True, cfg_scale=3.0), 1.0, 1.0),
])
def test_ddim_round_matches_checker(op, kw, eta_q, eta_p):
    from paper_2411_11925_b200 import api
    from paper_2411_11925_b200.runner import DeviceRound
    wl = gen.Workload(**{**gen.WORKLOADS["tiny_fp32"].__dict__, **kw})
    inp = gen.make_round_inputs(wl)
    # a DDPM with ten times as many steps (linear beta) visited at T evenly spaced timesteps
    N = 10 * wl.T
    beta_full = gen.beta_linear(N)
    steps = np.linspace(N // wl.T, N, wl.T).astype(np.int64)
    inp.tfeat = np.ascontiguousarray(gen.timestep_features(N, wl.draft.F)[steps - 1])
    sq, sp = orc.ddim_schedule(beta_full, steps, eta_q), orc.ddim_schedule(beta_full, steps, eta_p)
    eq = orc.make_mlp_head(inp.w_q, inp.z_q, inp.tfeat, wl.cfg, wl.cfg_scale)
    ep = orc.make_mlp_head(inp.w_p, inp.z_p, inp.tfeat, wl.cfg, wl.cfg_scale)
    ref = orc.csd_round(eq, ep, sq, sp, inp.x_T, inp.eps, inp.u, inp.xi, inp.v, wl.B, wl.gamma, wl.cap)
    dr = DeviceRound(inp, coeffs_q=api.ddim_coefficients(beta_full, steps, eta_q),
                     coeffs_p=api.ddim_coefficients(beta_full, steps, eta_p))
    dr.fused_round()
    out = dr.results()
    st = compare_round(out, ref, wl, sq["sigma"][0], sp["sigma"][0], inp.u, inp.v, f"ddim {op}")
    print("ddim", op, kw, st)
    if eta_q != eta_p:
        assert abs(ref["log_sigma"]) > 1.0
    dr.ctx.close()


@pytest.mark.parametrize("eta", [1.0, 0.5])
def test_ddim_100_of_1000_steps_at_mar256_size_sampled_sequences(eta):
    # The sampler setting of the paper's DDIM table: 100 DDIM steps out of a 1000-step linear-beta ladder, at the
    # size and launch configuration of the benchmark's 256x256-shaped workload; the checker evaluates four sequences
    # (first, last, both sides of a 128-row tile boundary).
    from paper_2411_11925_b200 import api
    from paper_2411_11925_b200.runner import DeviceRound
    wl = gen.WORKLOADS["mar256"]
    inp = gen.make_round_inputs(wl)
    N = 1000
    beta_full = gen.beta_linear(N)
    steps = np.linspace(N // wl.T, N, wl.T).astype(np.int64)
    inp.tfeat = np.ascontiguousarray(gen.timestep_features(N, wl.draft.F)[steps - 1])
    co = api.ddim_coefficients(beta_full, steps, eta)
    dr = DeviceRound(inp, coeffs_q=co, coeffs_p=co)
    dr.fused_round()
    out = dr.results()
    assert np.all(np.isfinite(out["x0"])) and np.all(np.isfinite(out["logratio"]))
    seqs = [0, 15, 16, 63]
    sub = gen.select_sequences(inp, seqs)
    sched = orc.ddim_schedule(beta_full, steps, eta)
    eq = orc.make_mlp_head(sub.w_q, sub.z_q, sub.tfeat, wl.cfg, wl.cfg_scale)
    ep = orc.make_mlp_head(sub.w_p, sub.z_p, sub.tfeat, wl.cfg, wl.cfg_scale)
    ref = orc.csd_round(eq, ep, sched, sched, sub.x_T, sub.eps, sub.u, sub.xi, sub.v, len(seqs), wl.gamma, wl.cap)
    rows = sub.extras["rows"]
    gsub = {k: (out[k][rows] if out[k].shape[0] == wl.R else out[k][seqs]) for k in out if k != "cap_hits"}
    gsub["cap_hits"] = out["cap_hits"]
    st = compare_round(gsub, ref, sub.wl, sched["sigma"][0], sched["sigma"][0], sub.u, sub.v, f"ddim-100 eta {eta}", xi=sub.xi)
    print("ddim-100", eta, st)
    dr.ctx.close()
