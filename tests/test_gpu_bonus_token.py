"""GPU parity of the all-accepted branch of Alg. 1: the bonus token of position gamma + 1."""
import numpy as np
import pytest
import torch

from oracle import csd_oracle as orc
from paper_2411_11925_b200 import inputs as gen

from _parity import TOL_X

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("op,kw", [("f32", dict(B=7, gamma=4, T=10)),
                                   ("f16", dict(B=40, gamma=8, T=8, bf16=True, cfg=True, cfg_scale=3.0))])
def test_bonus_token_matches_checker_and_leaves_other_rows_alone(op, kw):
    from paper_2411_11925_b200.runner import DeviceRound
    wl = gen.Workload(**{**gen.WORKLOADS["tiny_fp32"].__dict__, **kw})
    inp = gen.make_round_inputs(wl)
    dr = DeviceRound(inp)
    # inputs of position gamma + 1: one row per sequence (two with guidance)
    nxt = gen.make_round_inputs(gen.Workload(**{**wl.__dict__, "gamma": 1}), seed_offset=321, weights=False)
    z_next = torch.from_numpy(nxt.z_p).to(dr.dev)
    x_T_next = torch.from_numpy(nxt.x_T).to(dr.dev)
    eps_next = torch.from_numpy(nxt.eps).to(dr.dev)
    # accepted counts chosen here (an input of the call): a mix of all-accepted and rejected sequences
    n = (np.arange(wl.B) % 3 != 1).astype(np.int32) * wl.gamma - (np.arange(wl.B) % 3 == 2).astype(np.int32)
    n_dev = torch.from_numpy(n).to(dr.dev)
    x_bonus = torch.full((wl.B, dr.C), -7.0, dtype=torch.float32, device=dr.dev)
    taken = torch.full((wl.B,), 9, dtype=torch.int32, device=dr.dev)
    for _ in range(2):
        dr.ctx.csd_bonus_token(dr.head_p, dr.sched_p, wl.B, wl.gamma, wl.cfg, wl.cfg_scale, z_next, x_T_next, eps_next,
                               n_dev, x_bonus, taken)
    dr.ctx.sync()
    sp = orc.ddpm_schedule(inp.beta, wl.tau)
    ep = orc.make_mlp_head(inp.w_p, nxt.z_p, inp.tfeat, wl.cfg, wl.cfg_scale)
    ref = orc.bonus_token(ep, sp, nxt.x_T, nxt.eps, n, wl.gamma)
    got, tk = x_bonus.cpu().numpy(), taken.cpu().numpy()
    np.testing.assert_array_equal(tk.astype(bool), ref["taken"])
    assert ref["taken"].any() and (~ref["taken"]).any()
    assert np.all(got[~ref["taken"]] == -7.0)
    err = float(np.max(np.abs(got[ref["taken"]] - ref["x_bonus"][ref["taken"]])))
    print("bonus token", op, "x err", err)
    assert err <= TOL_X[op]
    # the same rows through the plain target-only call give the same bits
    x0, mu1 = torch.zeros_like(x_bonus), torch.zeros_like(x_bonus)
    dr.ctx.csd_draft_denoise(dr.head_p, dr.sched_p, wl.B, wl.cfg, wl.cfg_scale, z_next, x_T_next, eps_next, x0, mu1, None)
    dr.ctx.sync()
    np.testing.assert_array_equal(got[ref["taken"]], x0.cpu().numpy()[ref["taken"]])
    dr.ctx.close()
