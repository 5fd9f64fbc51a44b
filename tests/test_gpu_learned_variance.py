"""GPU parity of the learned-variance calls (heads that predict the diagonal of Sigma_theta of Eq. 3; Sigma of Eq. 7
per token) against the float64 checker on the same seeded inputs."""
import math

import numpy as np
import pytest
import torch

from oracle import csd_oracle as orc
from paper_2411_11925_b200 import inputs as gen

from _parity import F32_EPS, TOL_LOGR, TOL_MU, TOL_X

pytestmark = pytest.mark.gpu

# lv = lv_min + (w + 1)/2 (lv_max - lv_min): the variance parameter w is an output projection like eps_hat and
# carries the same kind of error; half_logdet sums T * C / 2 of them
TOL_LV = {"f32": 1e-5, "f16": 2e-3, "bf16": 2e-2}


def _wl(**kw):
    base = dict(B=7, gamma=5, T=6, cfg=True, cfg_scale=2.5, bf16=False, operand="")
    base.update(kw)
    return gen.Workload(**{**gen.WORKLOADS["tiny_fp32"].__dict__, **base})


def _lv_spec(s):
    return gen.HeadSpec(s.L, s.W, s.Dz, s.C, s.F, var_out=True)


def _inputs(wl, close=0.0, identical=False):
    wl = gen.Workload(**{**wl.__dict__, "draft": _lv_spec(wl.draft), "target": _lv_spec(wl.target)})
    inp = gen.make_round_inputs(wl)
    if close > 0.0:
        rng = np.random.default_rng(31)
        inp.w_q = gen.perturb_head_weights(inp.w_p, rng, close, wl.bf16)
        inp.z_q = inp.z_p
    if identical:
        inp.w_q, inp.z_q = inp.w_p, inp.z_p
    return inp


class LvRound:
    def __init__(self, inp, tau_q=1.0, tau_p=1.0):
        from paper_2411_11925_b200 import api
        wl = inp.wl
        self.inp, self.wl = inp, wl
        self.dev = torch.device("cuda", 0)
        self.ctx = api.Context(0)
        op = wl.operand_format
        self.hq = api.Head(self.ctx, inp.w_q, op, var_out=True)
        self.hp = api.Head(self.ctx, inp.w_p, op, var_out=True)
        self.tfeat = torch.from_numpy(inp.tfeat).to(self.dev)
        cq, cp = api.lv_ddpm_coefficients(inp.beta, tau_q), api.lv_ddpm_coefficients(inp.beta, tau_p)
        self.sq = api.ScheduleLV(cq["a"], cq["b"], cq["lv_min"], cq["lv_max"], self.tfeat)
        self.sp = api.ScheduleLV(cp["a"], cp["b"], cp["lv_min"], cp["lv_max"], self.tfeat)
        to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(self.dev)
        self.z_q, self.z_p, self.x_T, self.eps = to(inp.z_q), to(inp.z_p), to(inp.x_T), to(inp.eps)
        self.u, self.xi, self.v = to(inp.u), to(inp.xi), to(inp.v)
        B, R, C = wl.B, wl.R, wl.draft.C
        f = dict(dtype=torch.float32, device=self.dev)
        for n in ("x0", "mu1_q", "lv1_q", "mu1_p", "lv1_p"):
            setattr(self, n, torch.zeros(R, C, **f))
        for n in ("hld_q", "hld_p", "log_sigma_rows"):
            setattr(self, n, torch.zeros(R, **f))
        self.logratio = torch.zeros(B, wl.gamma, **f)
        self.x_new = torch.zeros(B, C, **f)
        for n in ("n_accept", "accept_mask", "n_prop", "flags"):
            setattr(self, n, torch.zeros(B, dtype=torch.int32, device=self.dev))
        self.cap_hits = torch.zeros(1, dtype=torch.int32, device=self.dev)

    def three_calls(self):
        wl, c = self.wl, self.ctx
        C = wl.draft.C
        c.csd_draft_denoise_lv(self.hq, self.sq, wl.R, wl.cfg, wl.cfg_scale, self.z_q, self.x_T, self.eps, self.x0,
                               self.mu1_q, self.lv1_q, self.hld_q, None)
        c.csd_verify_lv(self.hp, self.sp, wl.B, wl.gamma, wl.cfg, wl.cfg_scale, self.z_p, self.x_T, self.eps, self.x0,
                        self.mu1_q, self.lv1_q, self.hld_q, self.u, self.logratio, self.n_accept, self.accept_mask,
                        self.mu1_p, self.lv1_p, self.hld_p, self.log_sigma_rows)
        c.csd_resample_lv(wl.B, wl.gamma, C, wl.cap, self.log_sigma_rows, self.n_accept, self.mu1_p, self.lv1_p,
                          self.mu1_q, self.lv1_q, self.xi, self.v, self.x_new, self.n_prop, self.flags, self.cap_hits)

    def fused(self):
        wl = self.wl
        self.ctx.csd_round_lv(self.hq, self.hp, self.sq, self.sp, wl.B, wl.gamma, wl.cfg, wl.cfg_scale, wl.cap, self.z_q,
                              self.z_p, self.x_T, self.eps, self.u, self.xi, self.v, self.x0, self.mu1_q, self.lv1_q,
                              self.hld_q, self.mu1_p, self.lv1_p, self.hld_p, self.log_sigma_rows, self.logratio,
                              self.n_accept, self.accept_mask, self.x_new, self.n_prop, self.flags, self.cap_hits)

    NAMES = ("x0", "mu1_q", "lv1_q", "mu1_p", "lv1_p", "hld_q", "hld_p", "log_sigma_rows", "logratio", "n_accept",
             "accept_mask", "x_new", "n_prop", "flags", "cap_hits")

    def results(self):
        self.ctx.sync()
        return {n: getattr(self, n).cpu().numpy().copy() for n in self.NAMES}


def _ref(inp, tau_q=1.0, tau_p=1.0):
    wl = inp.wl
    sq, sp = orc.lv_schedule(inp.beta, tau_q), orc.lv_schedule(inp.beta, tau_p)
    fq = orc.make_mlp_head_lv(inp.w_q, inp.z_q, inp.tfeat, wl.cfg, wl.cfg_scale)
    fp = orc.make_mlp_head_lv(inp.w_p, inp.z_p, inp.tfeat, wl.cfg, wl.cfg_scale)
    return orc.csd_round_lv(fq, fp, sq, sp, inp.x_T, inp.eps, inp.u, inp.xi, inp.v, wl.B, wl.gamma, wl.cap)


def _eq8_diag(g):
    """Eq. 7/8 with diagonal covariances written out in float64 on the GPU's own arrays."""
    x0, mq, lq, mp, lp = (g[k].astype(np.float64) for k in ("x0", "mu1_q", "lv1_q", "mu1_p", "lv1_p"))
    nq = np.sum(0.5 * lq + 0.5 * (x0 - mq) ** 2 * np.exp(-lq), axis=1)
    npp = np.sum(0.5 * lp + 0.5 * (x0 - mp) ** 2 * np.exp(-lp), axis=1)
    return g["hld_q"].astype(np.float64) - g["hld_p"].astype(np.float64) + nq - npp, np.abs(nq) + np.abs(npp)


def _compare(g, ref, wl, u, rows=None, seqs=None, label=""):
    op = wl.operand_format
    T = wl.T
    C = ref["x0"].shape[1]
    sel = (lambda a: a) if rows is None else (lambda a: a[rows] if a.shape[0] == g["x0"].shape[0] else a[seqs])
    gs = {k: sel(v) for k, v in g.items() if k != "cap_hits"}
    st = {}
    for k, rk in (("x0", "x0"), ("mu1_q", "mu1_q"), ("mu1_p", "mu1_p")):
        st[k] = float(np.max(np.abs(gs[k] - ref[rk])))
        assert st[k] <= TOL_X[op], (label, st)
    for k in ("lv1_q", "lv1_p"):
        st[k] = float(np.max(np.abs(gs[k] - ref[k])))
        assert st[k] <= TOL_LV[op], (label, st)
    for k, rk in (("hld_q", "half_logdet_q"), ("hld_p", "half_logdet_p")):
        st[k] = float(np.max(np.abs(gs[k] - ref[rk])))
        assert st[k] <= TOL_LV[op] * 0.5 * C * max(1, T - 1) + 2e-6 * np.abs(ref[rk]).max(), (label, st)
    np.testing.assert_allclose(gs["log_sigma_rows"], gs["hld_q"] - gs["hld_p"], rtol=0, atol=1e-5 * (1 + np.abs(gs["hld_q"]).max()))
    # the ratio kernel against Eq. 7/8 on the GPU's own arrays
    own, mag = _eq8_diag(gs)
    lr = gs["logratio"].astype(np.float64)
    st["logr_kernel_err"] = float(np.max(np.abs(lr.reshape(-1) - own)))
    assert np.all(np.abs(lr.reshape(-1) - own) <= TOL_LOGR + 16 * F32_EPS * (mag + np.abs(gs["hld_q"]) + np.abs(gs["hld_p"]))), (label, st)
    st["logr_err"] = float(np.max(np.abs(lr - ref["logratio"])))
    moderate = np.abs(ref["logratio"]) < 50
    st["logr_moderate_err"] = float(np.abs(lr - ref["logratio"])[moderate].max()) if moderate.any() else 0.0
    # decisions: the scan is integer work on the GPU's own log-ratio; against the checker a decision may flip only
    # if the log-ratio error reaches its margin
    logu32 = np.log(u.astype(np.float32)).astype(np.float32)
    gm = gs["accept_mask"].astype(np.int64) & 0xFFFFFFFF
    acc = ((gm[:, None] >> np.arange(wl.gamma)[None, :]) & 1).astype(bool)
    knife = np.abs(logu32.astype(np.float64) - lr) < 1e-5
    assert np.array_equal(acc | knife, (logu32 <= gs["logratio"]) | knife), label
    np.testing.assert_array_equal(gs["n_accept"], [(list(r) + [False]).index(False) for r in acc])
    logu = np.log(u.astype(np.float64))
    acc_ref = logu <= ref["logratio"]
    flipped = acc != acc_ref
    st["accept_mismatch"] = int(flipped.sum())
    st["accept_rate"] = float(acc_ref.mean())
    assert np.all(np.abs(ref["logratio"] - logu)[flipped] <= np.abs(lr - ref["logratio"])[flipped] + 1e-5), (label, st)
    same = np.all(acc == acc_ref, axis=1)
    np.testing.assert_array_equal(gs["n_accept"][same], ref["n_accept"][same])
    np.testing.assert_array_equal(gs["flags"][same] & 1, ref["flags"][same] & 1)
    sp = same & (ref["n_accept"] < wl.gamma) & (gs["n_prop"] == ref["n_prop"])
    st["resampled"], st["same_prop"] = int((same & (ref["n_accept"] < wl.gamma)).sum()), int(sp.sum())
    if sp.any():
        st["xnew_err"] = float(np.max(np.abs(gs["x_new"][sp] - ref["x_new"][sp])))
        assert st["xnew_err"] <= TOL_MU[op] + 1e-6, (label, st)
    print(label, st)
    return st


@pytest.mark.parametrize("op", ["f32", "f16", "bf16"])
def test_small_round_matches_checker_and_fused_round_matches_three_calls(op):
    # 2*7*5 = 70 head rows and 2*23*7 = 322 (three row tiles, ragged), W = 384: three column tiles, C = 16
    for kw in (dict(), dict(B=23, gamma=7, T=5, draft=gen.HeadSpec(1, 256, 128), target=gen.HeadSpec(2, 384, 192))):
        inp = _inputs(_wl(bf16=op != "f32", operand=op, **kw))
        r = LvRound(inp, 1.0, 0.95)
        r.three_calls()
        a = r.results()
        _compare(a, _ref(inp, 1.0, 0.95), inp.wl, inp.u, label=f"lv {op} {kw}")
        r.fused()
        b = r.results()
        for k in LvRound.NAMES:
            np.testing.assert_array_equal(a[k], b[k], err_msg=k)
        r.ctx.close()


@pytest.mark.parametrize("op", ["f32", "f16"])
def test_close_heads_accept_reject_and_resample_with_predicted_variances(op):
    inp = _inputs(_wl(B=48, gamma=8, T=10, cfg=False, bf16=op != "f32", operand=op,
                      draft=gen.HeadSpec(2, 256, 256), target=gen.HeadSpec(2, 256, 256)), close=1e-4)
    r = LvRound(inp)
    r.fused()
    st = _compare(r.results(), _ref(inp), inp.wl, inp.u, label=f"lv close {op}")
    assert 0.05 < st["accept_rate"] < 0.98 and st["resampled"] >= 5, st
    assert st["logr_moderate_err"] <= (5e-2 if op == "f32" else 0.25), st
    r.ctx.close()


@pytest.mark.parametrize("op", ["f32", "f16", "bf16"])
def test_identical_heads_give_exactly_zero_and_accept_everything(op):
    inp = _inputs(_wl(B=6, gamma=5, T=8, bf16=op != "f32", operand=op, draft=gen.HeadSpec(2, 256, 256)), identical=True)
    r = LvRound(inp)
    r.three_calls()
    g = r.results()
    assert np.all(g["logratio"] == 0.0) and np.all(g["log_sigma_rows"] == 0.0)
    assert np.all(g["n_accept"] == inp.wl.gamma) and np.all(g["flags"] == 0)
    np.testing.assert_array_equal(g["lv1_q"], g["lv1_p"])
    r.ctx.close()


def test_constant_variance_output_reproduces_the_fixed_variance_calls():
    # variance rows of Wout zero, their bias +1: lv = lv_max = log(tau^2 beta_t), i.e. the fixed-variance round
    from paper_2411_11925_b200.runner import DeviceRound
    wl = _wl(B=16, gamma=4, T=10, cfg=True, cfg_scale=2.0)
    inp = _inputs(wl, close=1e-4)
    C = inp.wl.draft.C
    for w in (inp.w_q, inp.w_p):
        w["Wout"] = w["Wout"].copy(); w["bout"] = w["bout"].copy()
        w["Wout"][C:] = 0.0; w["bout"][C:] = 1.0
    r = LvRound(inp, 0.9, 0.9)
    r.three_calls()
    g = r.results()
    import dataclasses
    cut = lambda w: {**w, "Wout": np.ascontiguousarray(w["Wout"][:C]), "bout": np.ascontiguousarray(w["bout"][:C])}
    fixed = dataclasses.replace(inp, wl=wl, w_q=cut(inp.w_q), w_p=cut(inp.w_p))     # same z, noise and uniforms
    dr = DeviceRound(fixed, tau_q=0.9, tau_p=0.9)
    dr.three_calls()
    f = dr.results()
    for k in ("x0", "mu1_q", "mu1_p"):
        assert np.max(np.abs(g[k] - f[k])) <= 2e-6, k
    assert np.max(np.abs(g["logratio"] - f["logratio"])) <= 5e-2
    margin = np.abs(f["logratio"] - np.log(inp.u))
    ok = np.all(margin > 5e-2, axis=1)
    np.testing.assert_array_equal(g["n_accept"][ok], f["n_accept"][ok])
    assert np.max(np.abs(g["log_sigma_rows"])) <= 1e-4
    dr.ctx.close(); r.ctx.close()


def test_mar256_shaped_round_sampled_sequences():
    # B=64, gamma=8, T=100, guidance, 3x1024 and 6x1024 heads with 32 output columns; the checker evaluates the
    # first and last sequence and both sides of a 128-row tile boundary
    inp = _inputs(gen.WORKLOADS["mar256"])
    wl = inp.wl
    r = LvRound(inp)
    r.fused()
    g = r.results()
    assert np.all(np.isfinite(g["x0"])) and np.all(np.isfinite(g["logratio"]))
    seqs = [0, 15, 16, 63]
    sub = gen.select_sequences(inp, seqs)
    _compare(g, _ref(sub), sub.wl, sub.u, rows=sub.extras["rows"], seqs=seqs, label="lv mar256-shaped")
    r.fused()
    again = r.results()
    for k in LvRound.NAMES:
        np.testing.assert_array_equal(g[k], again[k], err_msg=k)
    r.ctx.close()


def test_fixed_and_learned_variance_calls_reject_the_other_kind_of_head():
    from paper_2411_11925_b200 import api
    inp = _inputs(_wl(B=2))
    r = LvRound(inp)
    sched = api.Schedule(r.sq.a, r.sq.b, np.full(inp.wl.T, 0.1, np.float32), r.tfeat)
    with pytest.raises(api.CsdError) as e:
        r.ctx.csd_draft_denoise(r.hq, sched, inp.wl.R, inp.wl.cfg, inp.wl.cfg_scale, r.z_q, r.x_T, r.eps, r.x0, r.mu1_q)
    assert e.value.code == -3
    r.ctx.sync()
    r.ctx.close()
