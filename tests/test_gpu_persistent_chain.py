"""The persistent chain kernel (one launch per chain when a layer is one wave of 128 x 128 tiles and W = 1024): whole
rounds against the float64 checker, against the three-kernel layer layout, fused against separate calls, with guidance
and without, ragged token counts, both operand formats, one-block and several-block heads."""
import numpy as np
import pytest

from oracle import csd_oracle as orc
from paper_2411_11925_b200 import inputs as gen

from _parity import TOL_X, compare_round

pytestmark = pytest.mark.gpu


def _wl(**kw):
    base = dict(B=64, gamma=4, T=4, bf16=True, cfg=True, cfg_scale=3.0, draft=gen.HeadSpec(1, 1024, 256),
                target=gen.HeadSpec(2, 1024, 256))
    base.update(kw)
    return gen.Workload(**{**gen.WORKLOADS["tiny_fp32"].__dict__, **base})


def _ref(inp):
    wl = inp.wl
    s = orc.ddpm_schedule(inp.beta, wl.tau)
    eq = orc.make_mlp_head(inp.w_q, inp.z_q, inp.tfeat, wl.cfg, wl.cfg_scale)
    ep = orc.make_mlp_head(inp.w_p, inp.z_p, inp.tfeat, wl.cfg, wl.cfg_scale)
    return orc.csd_round(eq, ep, s, s, inp.x_T, inp.eps, inp.u, inp.xi, inp.v, wl.B, wl.gamma, wl.cap), float(s["sigma"][0])


@pytest.mark.parametrize("op,kw", [
    ("f16", dict()),                                                          # 256 tokens with guidance: 4 row blocks
    ("bf16", dict(operand="bf16", cfg=False, cfg_scale=1.0, gamma=8, T=3,     # 512 tokens, no guidance: 4 row blocks
                  draft=gen.HeadSpec(2, 1024, 128), target=gen.HeadSpec(2, 1024, 128))),
    ("f16", dict(B=47, gamma=8, T=3)),                                        # 376 tokens: 6 row blocks, the last one ragged
    ("f16", dict(B=40, gamma=8, T=3)),                                        # 320 tokens: 5 row blocks, paired with an empty sixth
    ("f16", dict(T=1)),                                                       # a single denoising step
    ("f16", dict(B=121, gamma=4, T=2, cfg=False, cfg_scale=1.0,               # 484 tokens without guidance: ragged last block
                 draft=gen.HeadSpec(1, 1024, 128), target=gen.HeadSpec(3, 1024, 128))),
])
def test_persistent_chain_round_matches_checker_and_the_plain_layers(op, kw):
    from paper_2411_11925_b200 import api
    from paper_2411_11925_b200.runner import DeviceRound
    inp = gen.make_round_inputs(_wl(**kw))
    dr = DeviceRound(inp)
    dr.ctx.set_wait_limit(400_000_000)       # a stuck wait ends after a fifth of a second
    l0 = dr.ctx.launch_count()
    dr.three_calls()
    a = dr.results()
    launches = dr.ctx.launch_count() - l0
    assert launches < 30, launches           # two chains of one kernel each (plus their set-up), not 2 T (2L + 3)
    ref, s1 = _ref(inp)
    st = compare_round(a, ref, inp.wl, s1, s1, inp.u, inp.v, f"persistent chain {op} {kw}", xi=inp.xi)
    print("persistent chain", op, kw, {k: st[k] for k in ("x0_err", "mu1p_err", "logr_err_over_tol")}, "launches", launches)
    # the fused round launches the same two kernels side by side: same bits; and so does a repeat
    dr.fused_round()
    b = dr.results()
    dr.three_calls()
    c = dr.results()
    for k in ("x0", "mu1_q", "mu1_p", "logratio", "n_accept", "accept_mask", "x_new", "n_prop", "flags"):
        np.testing.assert_array_equal(a[k], b[k], err_msg=f"fused {k}")
        np.testing.assert_array_equal(a[k], c[k], err_msg=f"repeat {k}")
    # the three-kernel layer layout computes the same function with other roundings
    dr.ctx.set_chain_mode(api.Context.CHAIN_LAYERS_PLAIN)
    l1 = dr.ctx.launch_count()
    dr.three_calls()
    assert dr.ctx.launch_count() - l1 > 2 * inp.wl.T * 5
    d = dr.results()
    for k in ("x0", "mu1_q", "mu1_p"):
        assert float(np.max(np.abs(a[k] - d[k]))) <= TOL_X[op] / (2 if op == "bf16" else 4), k
    dr.ctx.set_wait_limit(0)
    dr.ctx.close()


def test_identical_heads_give_exactly_zero_in_the_persistent_chain():
    from paper_2411_11925_b200.runner import DeviceRound
    inp = gen.make_round_inputs(_wl(B=32, gamma=8, T=5, draft=gen.HeadSpec(2, 1024, 256), target=gen.HeadSpec(2, 1024, 256)))
    inp.w_q, inp.z_q = inp.w_p, inp.z_p
    dr = DeviceRound(inp)
    l0 = dr.ctx.launch_count()
    dr.fused_round()
    out = dr.results()
    assert dr.ctx.launch_count() - l0 < 30
    assert np.all(out["logratio"] == 0.0)
    assert np.all(out["n_accept"] == inp.wl.gamma) and np.all(out["flags"] == 0)
    np.testing.assert_array_equal(out["mu1_q"], out["mu1_p"])
    dr.ctx.close()


def test_recorded_trajectory_is_the_chain_itself():
    # csd_draft_denoise_traj through the persistent kernel: the records' last slots are the call's outputs, every
    # recorded state is the recorded mean plus the step's noise, and the plain call returns the same bits
    import torch
    from paper_2411_11925_b200 import api
    from paper_2411_11925_b200.runner import DeviceRound
    inp = gen.make_round_inputs(_wl(B=32, gamma=8, T=6))
    dr = DeviceRound(inp)
    wl = inp.wl
    l0 = dr.ctx.launch_count()
    dr.draft_traj()
    dr.ctx.sync()
    assert dr.ctx.launch_count() - l0 < 15
    tx, tm = dr.traj_x.cpu().numpy(), dr.traj_mu.cpu().numpy()
    np.testing.assert_array_equal(tx[0], inp.x_T.astype(np.float32))
    sig = api.ddpm_coefficients(inp.beta, wl.tau)["sigma"]
    for j in range(wl.T):
        t = wl.T - j
        want = tm[j].astype(np.float64) + float(sig[t - 1]) * inp.eps[t - 1].astype(np.float64)
        assert float(np.max(np.abs(tx[j + 1] - want))) <= 2e-6 * max(1.0, float(np.abs(tx[j + 1]).max()))
    dr.draft()
    dr.ctx.sync()
    np.testing.assert_array_equal(dr.x0.cpu().numpy(), tx[-1])
    np.testing.assert_array_equal(dr.mu1_q.cpu().numpy(), tm[-1])
    dr.ctx.close()
