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


@pytest.mark.parametrize("op", ["f32", "f16"])
def test_bonus_rows_folded_into_the_verify_chain_match_the_two_call_form(op):
    # csd_verify_bonus / csd_round_bonus run the B rows of position gamma + 1 as rows R..R+B of the verifying chain.
    # Close heads with a shared condition vector, so that some sequences accept all gamma drafts and others do not.
    from paper_2411_11925_b200 import api
    from paper_2411_11925_b200.runner import DeviceRound
    wl = gen.Workload(**{**gen.WORKLOADS["tiny_fp32"].__dict__, "B": 48, "gamma": 4, "T": 8, "bf16": op != "f32",
                         "operand": op, "cfg": True, "cfg_scale": 2.0, "perturb_std": 1e-4,
                         "draft": gen.HeadSpec(2, 256, 256), "target": gen.HeadSpec(2, 256, 256)})
    inp = gen.make_round_inputs(wl)
    inp.z_q = inp.z_p
    dr = DeviceRound(inp)
    nxt = gen.make_round_inputs(gen.Workload(**{**wl.__dict__, "gamma": 1}), seed_offset=321, weights=False)
    z_next, x_T_next, eps_next = (torch.from_numpy(a).to(dr.dev) for a in (nxt.z_p, nxt.x_T, nxt.eps))
    keys = ("logratio", "n_accept", "accept_mask", "mu1_p")

    def two_calls():
        xb = torch.full((wl.B, dr.C), -7.0, dtype=torch.float32, device=dr.dev)
        tk = torch.full((wl.B,), 9, dtype=torch.int32, device=dr.dev)
        dr.draft(); dr.verify()
        dr.ctx.csd_bonus_token(dr.head_p, dr.sched_p, wl.B, wl.gamma, wl.cfg, wl.cfg_scale, z_next, x_T_next, eps_next,
                               dr.n_accept, xb, tk)
        dr.resample()
        out = dr.results()
        return out, xb.cpu().numpy(), tk.cpu().numpy()

    def fused_verify():
        xb = torch.full((wl.B, dr.C), -7.0, dtype=torch.float32, device=dr.dev)
        tk = torch.full((wl.B,), 9, dtype=torch.int32, device=dr.dev)
        dr.draft()
        dr.ctx.csd_verify_bonus(dr.head_p, dr.sched_p, dr.sched_q, wl.B, wl.gamma, wl.cfg, wl.cfg_scale, dr.z_p, dr.x_T,
                                dr.eps, dr.x0, dr.mu1_q, dr.u, z_next, x_T_next, eps_next, dr.logratio, dr.n_accept,
                                dr.accept_mask, dr.mu1_p, xb, tk)
        dr.resample()
        out = dr.results()
        return out, xb.cpu().numpy(), tk.cpu().numpy()

    def fused_round():
        xb = torch.full((wl.B, dr.C), -7.0, dtype=torch.float32, device=dr.dev)
        tk = torch.full((wl.B,), 9, dtype=torch.int32, device=dr.dev)
        dr.ctx.csd_round_bonus(dr.head_q, dr.head_p, dr.sched_q, dr.sched_p, wl.B, wl.gamma, wl.cfg, wl.cfg_scale, wl.cap,
                               dr.z_q, dr.z_p, dr.x_T, dr.eps, dr.u, dr.xi, dr.v, z_next, x_T_next, eps_next, dr.x0,
                               dr.mu1_q, dr.mu1_p, dr.logratio, dr.n_accept, dr.accept_mask, dr.x_new, dr.n_prop, dr.flags,
                               dr.cap_hits, xb, tk)
        out = dr.results()
        return out, xb.cpu().numpy(), tk.cpu().numpy()

    for mode in (api.Context.CHAIN_LAYERS_PLAIN, api.Context.CHAIN_LAYERS):
        dr.ctx.set_chain_mode(mode)
        a, xa, ta = two_calls()
        b, xb_, tb = fused_verify()
        c, xc, tc = fused_round()
        assert 0 < ta.sum() < wl.B, ta                        # both branches of Alg. 1 occur
        assert np.all(xa[ta == 0] == -7.0) and np.all(xb_[tb == 0] == -7.0)
        # the round is the three calls with the same row counts: same bits in either layout
        for k in keys + ("x0", "mu1_q", "x_new", "n_prop", "flags"):
            np.testing.assert_array_equal(b[k], c[k], err_msg=f"round vs calls {k}")
        np.testing.assert_array_equal(xb_, xc); np.testing.assert_array_equal(tb, tc)
        if mode == api.Context.CHAIN_LAYERS_PLAIN:
            for k in keys:
                np.testing.assert_array_equal(a[k], b[k], err_msg=k)
            np.testing.assert_array_equal(xa, xb_); np.testing.assert_array_equal(ta, tb)
        else:
            assert np.max(np.abs(a["mu1_p"] - b["mu1_p"])) <= TOL_X[op] / 4
            both = (ta == 1) & (tb == 1)
            assert np.max(np.abs(xa[both] - xb_[both])) <= TOL_X[op] / 4
    # against the checker: the bonus rows are ordinary target samples
    sp = orc.ddpm_schedule(inp.beta, wl.tau)
    ref = orc.bonus_token(orc.make_mlp_head(inp.w_p, nxt.z_p, inp.tfeat, wl.cfg, wl.cfg_scale), sp, nxt.x_T, nxt.eps,
                          b["n_accept"], wl.gamma)
    np.testing.assert_array_equal(tb.astype(bool), ref["taken"])
    assert np.max(np.abs(xb_[ref["taken"]] - ref["x_bonus"][ref["taken"]])) <= TOL_X[op]
    dr.ctx.close()
