"""The persistent small-batch chain kernel (CSD_CHAIN_SMALL_BATCH): chains of at most 128 head rows, the calling
pattern of Alg. 1's draft loop (x_i ~ q_i one position at a time), against the float64 checker and against the
layer kernels."""
import numpy as np
import pytest
import torch

from oracle import csd_oracle as orc
from paper_2411_11925_b200 import inputs as gen

from _parity import TOL_X, compare_round

pytestmark = pytest.mark.gpu


def _wl(**kw):
    base = dict(B=8, gamma=4, T=6, bf16=True, cfg=True, cfg_scale=3.0, draft=gen.HeadSpec(2, 512, 128),
                target=gen.HeadSpec(3, 512, 256))
    base.update(kw)
    return gen.Workload(**{**gen.WORKLOADS["tiny_fp32"].__dict__, **base})


def _round(inp, mode):
    from paper_2411_11925_b200.runner import DeviceRound
    dr = DeviceRound(inp)
    dr.ctx.set_wait_limit(400_000_000)       # a stuck wait ends after a fifth of a second
    dr.ctx.set_chain_mode(mode)
    return dr


def _ref(inp):
    wl = inp.wl
    s = orc.ddpm_schedule(inp.beta, wl.tau)
    eq = orc.make_mlp_head(inp.w_q, inp.z_q, inp.tfeat, wl.cfg, wl.cfg_scale)
    ep = orc.make_mlp_head(inp.w_p, inp.z_p, inp.tfeat, wl.cfg, wl.cfg_scale)
    return orc.csd_round(eq, ep, s, s, inp.x_T, inp.eps, inp.u, inp.xi, inp.v, wl.B, wl.gamma, wl.cap), float(s["sigma"][0])


@pytest.mark.parametrize("op,kw", [
    ("f16", dict()),                                               # 64 head rows, W = 512 (one k-block per K slice)
    ("bf16", dict(operand="bf16")),
    ("f16", dict(B=16, gamma=4, cfg=True)),                        # exactly 128 head rows
    ("f16", dict(B=37, gamma=3, cfg=False, cfg_scale=1.0)),        # 111 rows: ragged, no guidance
    ("f16", dict(B=1, gamma=1, T=1, cfg=False, cfg_scale=1.0)),    # one row, one step
    ("f16", dict(B=5, gamma=4, T=5, draft=gen.HeadSpec(1, 1024, 256), target=gen.HeadSpec(2, 1536, 128))),  # two / three k-blocks per slice
])
def test_small_batch_round_matches_checker_and_the_layer_kernels(op, kw):
    from paper_2411_11925_b200 import api
    inp = gen.make_round_inputs(_wl(**kw))
    dr = _round(inp, api.Context.CHAIN_SMALL_BATCH)
    l0 = dr.ctx.launch_count()
    dr.three_calls()
    a = dr.results()
    launches = dr.ctx.launch_count() - l0
    assert launches < 30, launches                                  # two chains of one kernel each, not 2 T (2L + 3)
    ref, s1 = _ref(inp)
    st = compare_round(a, ref, inp.wl, s1, s1, inp.u, inp.v, f"small batch {op} {kw}", xi=inp.xi)
    print("small batch", op, kw, {k: st[k] for k in ("x0_err", "mu1p_err", "logr_err_over_tol")}, "launches", launches)
    # the fused round runs the same two kernels one after the other: same bits; and so does a repeat
    dr.fused_round()
    b = dr.results()
    dr.three_calls()
    c = dr.results()
    for k in ("x0", "mu1_q", "mu1_p", "logratio", "n_accept", "accept_mask", "x_new", "n_prop", "flags"):
        np.testing.assert_array_equal(a[k], b[k], err_msg=f"fused {k}")
        np.testing.assert_array_equal(a[k], c[k], err_msg=f"repeat {k}")
    # the layer kernels compute the same function with other roundings
    dr.ctx.set_chain_mode(api.Context.CHAIN_LAYERS)
    dr.three_calls()
    d = dr.results()
    for k in ("x0", "mu1_q", "mu1_p"):
        assert float(np.max(np.abs(a[k] - d[k]))) <= TOL_X[op] / (2 if op == "bf16" else 4), k   # both carry their own rounding
    dr.ctx.set_wait_limit(0)
    dr.ctx.close()


def test_identical_heads_give_exactly_zero_in_small_batch_mode():
    from paper_2411_11925_b200 import api
    inp = gen.make_round_inputs(_wl(B=6, gamma=5, T=8, draft=gen.HeadSpec(2, 512, 256), target=gen.HeadSpec(2, 512, 256)))
    inp.w_q, inp.z_q = inp.w_p, inp.z_p
    dr = _round(inp, api.Context.CHAIN_SMALL_BATCH)
    dr.three_calls()
    out = dr.results()
    assert np.all(out["logratio"] == 0.0) and np.all(out["n_accept"] == inp.wl.gamma)
    dr.ctx.set_wait_limit(0)
    dr.ctx.close()


def test_sequential_draft_calls_at_benchmark_size():
    # one position of the 256x256-shaped workload: 64 sequences x 2 guidance halves = 128 head rows of the 3 x 1024
    # draft head, T = 100; the checker evaluates the first and the last sequence
    from paper_2411_11925_b200 import api
    wl = gen.Workload(**{**gen.WORKLOADS["mar256"].__dict__, "gamma": 1})
    inp = gen.make_round_inputs(wl)
    dr = _round(inp, api.Context.CHAIN_SMALL_BATCH)
    dr.draft()
    dr.ctx.sync()
    x0 = dr.x0.cpu().numpy()
    sub = gen.select_sequences(inp, [0, 63])
    s = orc.ddpm_schedule(inp.beta, wl.tau)
    ref = orc.denoise(orc.make_mlp_head(sub.w_q, sub.z_q, sub.tfeat, wl.cfg, wl.cfg_scale), s, sub.x_T, sub.eps)
    err = float(np.max(np.abs(x0[sub.extras["rows"]] - ref["x0"])))
    print("sequential draft call, small-batch kernel: x0 err", err)
    assert err <= TOL_X["f16"]
    dr.draft()
    dr.ctx.sync()
    np.testing.assert_array_equal(x0, dr.x0.cpu().numpy())
    dr.ctx.set_wait_limit(0)
    dr.ctx.close()
