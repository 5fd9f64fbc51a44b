"""GPU parity of the Gaussian-mixture head calls (explicit p and q) against the float64 checker."""
import numpy as np
import pytest
import torch

from oracle import csd_oracle as orc

pytestmark = pytest.mark.gpu


def _case(seed, B, gamma, Kq, Kp, C, cap, close):
    rng = np.random.default_rng(seed)
    R = B * gamma
    mix = lambda K: (rng.standard_normal((R, K)).astype(np.float32), rng.standard_normal((R, K, C)).astype(np.float32),
                     (0.3 * rng.standard_normal((R, K, C)) - 0.5).astype(np.float32))
    p = mix(Kp)
    if close:        # draft = target with perturbed parameters: ratios of order one
        q = tuple((a + close * rng.standard_normal(a.shape)).astype(np.float32) for a in p)
    else:
        q = mix(Kq)
    f = lambda *s: rng.random(s).astype(np.float32).clip(1e-6, 1 - 1e-6)
    g = lambda *s: rng.standard_normal(s).astype(np.float32)
    return dict(q=q, p=p, u_comp=f(R), noise=g(R, C), u=f(B, gamma), w=f(B, cap), xi=g(B, cap, C), v=f(B, cap))


@pytest.mark.parametrize("B,gamma,Kq,Kp,C,cap,close", [(37, 8, 4, 4, 16, 16, 0.05), (5, 32, 3, 7, 16, 8, 0.0),
                                                       (64, 4, 1, 1, 1, 32, 0.3), (9, 1, 5, 5, 32, 4, 0.02)])
def test_gmm_round_matches_checker(B, gamma, Kq, Kp, C, cap, close):
    from paper_2411_11925_b200 import api
    d = _case(11, B, gamma, Kq, Kp, C, cap, close)
    dev = torch.device("cuda", 0)
    ctx = api.Context(0)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    q, p = tuple(t(a) for a in d["q"]), tuple(t(a) for a in d["p"])
    R = B * gamma
    x = torch.zeros(R, C, device=dev); comp = torch.zeros(R, dtype=torch.int32, device=dev)
    lr = torch.zeros(B, gamma, device=dev)
    n_acc, mask, n_prop, flags = (torch.zeros(B, dtype=torch.int32, device=dev) for _ in range(4))
    x_new = torch.full((B, C), 7.0, device=dev); hits = torch.full((1,), 99, dtype=torch.int32, device=dev)
    ctx.csd_gmm_draft_sample(R, C, q, t(d["u_comp"]), t(d["noise"]), x, comp)
    ctx.csd_gmm_verify(B, gamma, C, q, p, x, t(d["u"]), lr, n_acc, mask)
    ctx.csd_gmm_resample(B, gamma, C, cap, q, p, n_acc, t(d["w"]), t(d["xi"]), t(d["v"]), x_new, n_prop, flags, hits)
    ctx.sync()
    ref = orc.gmm_round(d["q"], d["p"], d["u_comp"], d["noise"], d["u"], d["w"], d["xi"], d["v"], B, gamma, cap)
    # component choice: exact except where u sits on a boundary of the cumulative weights (fp32 vs float64 sums)
    wq = np.exp(d["q"][0].astype(np.float64)); wq /= wq.sum(1, keepdims=True)
    near = np.min(np.abs(np.cumsum(wq, 1) - d["u_comp"][:, None].astype(np.float64)), axis=1) < 1e-5
    gc = comp.cpu().numpy()
    np.testing.assert_array_equal(gc[~near], ref["comp"][~near])
    same_c = gc == ref["comp"]
    gx = x.cpu().numpy()
    assert np.max(np.abs(gx[same_c] - ref["x"][same_c])) <= 1e-5
    # log-ratio: re-evaluate the checker at the GPU's own samples (rows whose component matched have the same x)
    want = (orc.gmm_logpdf(gx, *d["p"]) - orc.gmm_logpdf(gx, *d["q"])).reshape(B, gamma)
    glr = lr.cpu().numpy()
    scale = np.abs(orc.gmm_logpdf(gx, *d["p"])).reshape(B, gamma) + np.abs(orc.gmm_logpdf(gx, *d["q"])).reshape(B, gamma)
    err = np.abs(glr - want)
    assert np.all(err <= 5e-4 + 4e-6 * scale), float(err.max())
    # decisions: integer work on the GPU's own log-ratio; against the checker a flip needs an error >= the margin
    gm = mask.cpu().numpy().astype(np.int64) & 0xFFFFFFFF
    acc = ((gm[:, None] >> np.arange(gamma)[None, :]) & 1).astype(bool)
    logu32 = np.log(d["u"]).astype(np.float32)
    knife = np.abs(logu32.astype(np.float64) - glr) < 1e-5
    assert np.array_equal(acc | knife, (logu32 <= glr) | knife)
    gn = n_acc.cpu().numpy()
    np.testing.assert_array_equal(gn, [(list(r) + [False]).index(False) for r in acc])
    acc_ref = np.log(d["u"].astype(np.float64)) <= want
    flipped = acc != acc_ref
    assert np.all(np.abs(want - np.log(d["u"].astype(np.float64)))[flipped] <= err[flipped] + 1e-5)
    # resampling, for sequences whose prefix length equals the checker's on the same samples
    n_ref, _ = orc.accept_prefix(want, d["u"])
    rs = orc.gmm_resample(gn, d["q"], d["p"], d["w"], d["xi"], d["v"], gamma, cap)
    gp, gf, gxn = n_prop.cpu().numpy(), flags.cpu().numpy(), x_new.cpu().numpy()
    np.testing.assert_array_equal(gf & 1, (gn < gamma).astype(gf.dtype))
    same = gp == rs["n_prop"]
    assert same.mean() > 0.95, same.mean()          # a threshold within rounding of v may flip a proposal
    np.testing.assert_array_equal(gf[same], rs["flags"][same])
    res = same & (gn < gamma)
    if res.any():
        assert np.max(np.abs(gxn[res] - rs["x_new"][res])) <= 1e-4
    assert np.all(gxn[gn == gamma] == 7.0) and np.all(gp[gn == gamma] == 0)
    assert int(hits.item()) == int(((gf & 2) != 0).sum())
    print("gmm", (B, gamma, Kq, Kp, C), "accept rate", float(acc_ref.mean()), "resampled", int((gn < gamma).sum()),
          "max logR err", float(err.max()), "n_prop agree", float(same.mean()))
    ctx.close()


def test_identical_mixtures_give_exactly_zero_on_the_gpu_and_bad_arguments_are_reported():
    from paper_2411_11925_b200 import api
    d = _case(5, 6, 5, 3, 3, 16, 4, 0.0)
    dev = torch.device("cuda", 0)
    ctx = api.Context(0)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    p = tuple(t(a) for a in d["p"])
    x = torch.zeros(30, 16, device=dev)
    ctx.csd_gmm_draft_sample(30, 16, p, t(d["u_comp"]), t(d["noise"]), x)
    lr = torch.ones(6, 5, device=dev); n = torch.zeros(6, dtype=torch.int32, device=dev)
    ctx.csd_gmm_verify(6, 5, 16, p, p, x, t(d["u"]), lr, n)
    ctx.sync()
    assert torch.all(lr == 0.0) and torch.all(n == 5)
    with pytest.raises(api.CsdError) as e:
        ctx.csd_gmm_verify(6, 33, 16, p, p, x, t(d["u"]), lr, n)
    assert e.value.code == -3
    with pytest.raises(api.CsdError) as e:
        ctx.csd_gmm_draft_sample(30, 40, p, t(d["u_comp"]), t(d["noise"]), x)
    assert e.value.code == -3
    ctx.sync()
    ctx.close()
