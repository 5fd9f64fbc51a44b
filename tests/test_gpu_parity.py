"""GPU parity: the CUDA library, called through its C ABI, against the float64 checker on the
same seeded inputs (element by element at sizes the checker finishes in seconds; sampled
sequences at the full benchmark size)."""
import numpy as np
import pytest
import torch

from oracle import csd_oracle as orc
from paper_2411_11925_b200 import inputs as gen

from _parity import TOL_X, compare_round

pytestmark = pytest.mark.gpu


def _wl(base="tiny_fp32", **kw):
    return gen.Workload(**{**gen.WORKLOADS[base].__dict__, **kw})


def _run(inp, fused=False, **kw):
    from paper_2411_11925_b200.runner import DeviceRound
    dr = DeviceRound(inp, **kw)
    dr.fused_round() if fused else dr.three_calls()
    out = dr.results()
    return dr, out


def _ref(inp, tau_q=None, tau_p=None):
    wl = inp.wl
    sq = orc.ddpm_schedule(inp.beta, wl.tau if tau_q is None else tau_q)
    sp = orc.ddpm_schedule(inp.beta, wl.tau if tau_p is None else tau_p)
    eq = orc.make_mlp_head(inp.w_q, inp.z_q, inp.tfeat, wl.cfg, wl.cfg_scale)
    ep = orc.make_mlp_head(inp.w_p, inp.z_p, inp.tfeat, wl.cfg, wl.cfg_scale)
    ref = orc.csd_round(eq, ep, sq, sp, inp.x_T, inp.eps, inp.u, inp.xi, inp.v, wl.B, wl.gamma, wl.cap)
    return ref, sq["sigma"][0], sp["sigma"][0]


def _check(inp, label, fused=False, tau_q=None, tau_p=None):
    dr, out = _run(inp, fused=fused, tau_q=tau_q, tau_p=tau_p)
    ref, s1q, s1p = _ref(inp, tau_q, tau_p)
    st = compare_round(out, ref, inp.wl, s1q, s1p, inp.u, inp.v, label, xi=inp.xi)
    print(label, st)
    dr.ctx.close()
    return st, out, ref


def test_tiny_fp32_workload_matches_checker():
    inp = gen.make_round_inputs(gen.WORKLOADS["tiny_fp32"])
    st, out, ref = _check(inp, "tiny_fp32")
    np.testing.assert_allclose(out["x1_q"], ref["x1_q"], atol=1e-4)


def test_fused_round_is_bit_identical_to_three_calls():
    for base, kw in (("tiny_fp32", dict(B=3, cfg=True, cfg_scale=2.0)),
                     ("tiny_fp32", dict(B=5, gamma=7, T=6, bf16=True, cfg=True, cfg_scale=3.0)),
                     ("tiny_fp32", dict(B=5, gamma=7, T=6, bf16=True, operand="bf16", cfg=True, cfg_scale=3.0)),
                     # 20 tiles of 128 columns per chain: alone a chain runs 64-wide tiles, side by side 128-wide
                     ("tiny_fp32", dict(B=80, gamma=8, T=3, bf16=True, cfg=True, cfg_scale=3.0,
                                        draft=gen.HeadSpec(1, 256, 128), target=gen.HeadSpec(2, 256, 128)))):
        inp = gen.make_round_inputs(_wl(base, **kw))
        dr, a = _run(inp, fused=False)
        dr.fused_round()
        b = dr.results()
        for k in ("x0", "mu1_q", "mu1_p", "logratio", "n_accept", "accept_mask", "x_new", "n_prop", "flags"):
            np.testing.assert_array_equal(a[k], b[k], err_msg=k)
        dr.ctx.close()


OPERANDS = ["f32", "bf16", "f16"]


@pytest.mark.parametrize("op", OPERANDS)
def test_identical_heads_give_zero_logratio_and_accept_all(op):
    wl = _wl(B=6, gamma=5, T=8, bf16=op != "f32", operand=op, cfg=True, cfg_scale=3.0, draft=gen.HeadSpec(2, 256, 256))
    inp = gen.make_round_inputs(wl)
    inp.w_q, inp.z_q = inp.w_p, inp.z_p
    dr, out = _run(inp)
    assert np.all(out["logratio"] == 0.0)
    assert np.all(out["n_accept"] == wl.gamma) and np.all(out["flags"] == 0) and np.all(out["n_prop"] == 0)
    np.testing.assert_array_equal(out["mu1_q"], out["mu1_p"])
    dr.ctx.close()


@pytest.mark.parametrize("op", OPERANDS)
def test_ragged_rows_guidance_and_several_tiles(op):
    # Rh = 2*B*gamma = 2*23*7 = 322 rows: three 128-row tensor-core tiles with a ragged tail (66 rows),
    # eleven 32-row tiles on the fp32 path with a 2-row tail; W = 384 gives three column tiles.
    wl = _wl(B=23, gamma=7, T=6, bf16=op != "f32", operand=op, cfg=True, cfg_scale=3.0,
             draft=gen.HeadSpec(1, 256, 128), target=gen.HeadSpec(2, 384, 192))
    _check(gen.make_round_inputs(wl), f"ragged {op}")


@pytest.mark.parametrize("op", OPERANDS)
def test_close_heads_exercise_accepts_rejects_and_resampling(op):
    # draft = target + small perturbation: log-ratios are O(1), so accepts, rejects and multi-proposal
    # resampling all occur and the 5e-2 tolerance is the binding one.
    wl = _wl(B=48, gamma=8, T=10, bf16=op != "f32", operand=op, cfg=False, perturb_std=1e-4,
             draft=gen.HeadSpec(2, 256, 256), target=gen.HeadSpec(2, 256, 256))
    inp = gen.make_round_inputs(wl)
    inp.z_q = inp.z_p                      # same condition vector: only the weights differ
    st, out, ref = _check(inp, f"close heads {op}", fused=True)
    assert 0.05 < st["accept_rate"] < 0.98, st
    assert st["resampled"] >= 5 and st["n_prop_max"] >= 2, st


def test_different_variances_exercise_the_sigma_term():
    # tau_q != tau_p: Sigma of Eq. 7 is not 1 and sigma_q,1 != sigma_p,1 (general form of Eq. 8)
    wl = _wl(B=16, gamma=4, T=10, perturb_std=1e-4, draft=gen.HeadSpec(2, 256, 256))
    inp = gen.make_round_inputs(wl)
    inp.z_q = inp.z_p
    st, out, ref = _check(inp, "sigma term", tau_q=1.0, tau_p=0.97)
    assert abs(ref["log_sigma"]) > 1.0


def test_accept_scan_kernel_all_masks_and_edge_cases():
    from paper_2411_11925_b200 import api
    dev = torch.device("cuda", 0)
    ctx = api.Context(0)
    rng = np.random.default_rng(5)
    for gamma in (1, 5, 8, 32):
        B, C = (2 ** gamma if gamma <= 8 else 300), 16
        R = B * gamma
        x0 = rng.standard_normal((R, C)).astype(np.float32)
        mu_q = (x0 + 0.01 * rng.standard_normal((R, C))).astype(np.float32)
        mu_p = (x0 + 0.012 * rng.standard_normal((R, C))).astype(np.float32)
        sp1, sq1, ls = 0.011, 0.01, 0.3
        lr = orc.log_ratio_closed(x0.astype(np.float64), mu_q.astype(np.float64), mu_p.astype(np.float64), sq1, sp1, ls)
        lr = lr.reshape(B, gamma)
        if gamma <= 8:      # every accept mask once: u just below / above the ratio
            bits = ((np.arange(B)[:, None] >> np.arange(gamma)[None, :]) & 1).astype(bool)
            u = np.where(bits, np.exp(lr - 0.5), np.exp(lr + 0.5))
            u = np.clip(u, 1e-30, None).astype(np.float32)
        else:
            u = rng.random((B, gamma)).astype(np.float32).clip(1e-7, 1)
        t = lambda a: torch.from_numpy(a).to(dev)
        d_lr = torch.zeros(B, gamma, device=dev); d_n = torch.zeros(B, dtype=torch.int32, device=dev)
        d_m = torch.zeros(B, dtype=torch.int32, device=dev)
        ctx.csd_accept_scan(B, gamma, C, ls, sp1, sq1, t(x0), t(mu_q), t(mu_p), t(u), d_lr, d_n, d_m)
        ctx.sync()
        g_lr = d_lr.cpu().numpy()
        np.testing.assert_allclose(g_lr, lr, atol=2e-3 + 1e-5 * np.abs(lr).max())
        n_ref, acc_ref = orc.accept_prefix(lr, u)
        near = np.abs(lr - np.log(u.astype(np.float64))) < 5e-2
        assert not near.any() or gamma > 8
        ok_rows = ~near.any(axis=1)
        np.testing.assert_array_equal(d_n.cpu().numpy()[ok_rows], n_ref[ok_rows])
        gm = d_m.cpu().numpy().astype(np.int64) & 0xFFFFFFFF
        accg = ((gm[:, None] >> np.arange(gamma)[None, :]) & 1).astype(bool)
        np.testing.assert_array_equal(accg[ok_rows], acc_ref[ok_rows])
    ctx.close()


def test_resample_kernel_matches_checker_including_cap_hits():
    from paper_2411_11925_b200 import api
    dev = torch.device("cuda", 0)
    ctx = api.Context(0)
    rng = np.random.default_rng(6)
    B, gamma, C, cap = 500, 6, 16, 8
    R = B * gamma
    mu_p = rng.standard_normal((R, C)).astype(np.float32)
    mu_q = (mu_p + 0.002 * rng.standard_normal((R, C))).astype(np.float32)   # low acceptance -> cap hits
    n_acc = rng.integers(0, gamma + 1, B).astype(np.int32)
    xi = rng.standard_normal((B, cap, C)).astype(np.float32)
    v = rng.random((B, cap)).astype(np.float32).clip(1e-7, 1 - 1e-7)
    sp1, sq1, ls = 0.01, 0.0105, -0.2
    ref = orc.resample(n_acc, mu_p.astype(np.float64), mu_q.astype(np.float64), sp1, sq1, ls, xi, v, gamma, cap)
    t = lambda a: torch.from_numpy(a).to(dev)
    x_new = torch.full((B, C), 7.0, device=dev)
    n_prop = torch.zeros(B, dtype=torch.int32, device=dev); flags = torch.zeros(B, dtype=torch.int32, device=dev)
    hits = torch.full((1,), 99, dtype=torch.int32, device=dev)
    for _ in range(2):       # second call: the cap-hit counter must restart from zero
        ctx.csd_resample(B, gamma, C, cap, ls, sp1, sq1, t(n_acc), t(mu_p), t(mu_q), t(xi), t(v), x_new, n_prop, flags, hits)
    ctx.sync()
    g_prop, g_flags, g_x = n_prop.cpu().numpy(), flags.cpu().numpy(), x_new.cpu().numpy()
    same = g_prop == ref["n_prop"]
    assert same.mean() > 0.97, same.mean()          # thresholds within rounding of v may flip a proposal
    np.testing.assert_array_equal(g_flags[same], ref["flags"][same])
    res = same & (n_acc < gamma)
    np.testing.assert_allclose(g_x[res], ref["x_new"][res], atol=1e-6)
    assert np.all(g_x[n_acc == gamma] == 7.0) and np.all(g_prop[n_acc == gamma] == 0)   # untouched
    assert ref["cap_hits"] > 10 and abs(int(hits.item()) - ref["cap_hits"]) <= (~same).sum()
    ctx.close()


def test_argument_errors_are_reported_not_raised_by_the_device():
    from paper_2411_11925_b200 import api
    ctx = api.Context(0)
    wl = _wl(B=2)
    inp = gen.make_round_inputs(wl)
    w_bad = dict(inp.w_p); w_bad["Wz"] = np.zeros((200, 256), np.float32)   # W = 200 not a multiple of 128
    with pytest.raises(api.CsdError) as e:
        api.Head(ctx, {**w_bad, "bz": np.zeros(200, np.float32)}, "f32")
    assert e.value.code == -3
    dev = torch.device("cuda", 0)
    z = torch.zeros(4, device=dev)
    with pytest.raises(api.CsdError) as e:
        ctx.csd_accept_scan(2, 33, 16, 0.0, 0.01, 0.01, z, z, z, z, z, z.int())
    assert e.value.code == -3 and "gamma" in str(e.value)
    with pytest.raises(api.CsdError) as e:
        ctx.csd_resample(2, 4, 16, 0, 0.0, 0.01, 0.01, z.int(), z, z, z, z, z, z.int(), z.int(), z.int())
    assert e.value.code == -1
    with pytest.raises(api.CsdError) as e:
        ctx.csd_accept_scan(2, 4, 16, 0.0, 0.01, 0.01, None, z, z, z, z, z.int())
    assert e.value.code == -1
    ctx.sync()
    ctx.close()


def _sampled(name, seqs, label):
    wl = gen.WORKLOADS[name]
    inp = gen.make_round_inputs(wl)
    dr, out = _run(inp, fused=True)
    sub = gen.select_sequences(inp, seqs)
    ref, s1q, s1p = _ref(sub)
    rows = sub.extras["rows"]
    gsub = {k: (out[k][rows] if out[k].shape[0] == wl.R else out[k][seqs]) for k in out if k != "cap_hits"}
    gsub["cap_hits"] = out["cap_hits"]
    st = compare_round(gsub, ref, sub.wl, s1q, s1p, sub.u, sub.v, label, xi=sub.xi)
    print(label, st)
    # properties that hold at any size: n_accept within [0, gamma], resampled exactly where n < gamma
    assert np.all((out["n_accept"] >= 0) & (out["n_accept"] <= wl.gamma))
    np.testing.assert_array_equal(out["flags"] & 1, (out["n_accept"] < wl.gamma).astype(out["flags"].dtype))
    assert np.all(np.isfinite(out["x0"])) and np.all(np.isfinite(out["logratio"]))
    assert int(out["cap_hits"][0]) == int(((out["flags"] & 2) != 0).sum())
    dr.ctx.close()
    return st


# Sampled sequences at full size: the first and the last sequence, both sides of the first 128-row tile boundary
# (row = b * gamma + i) and of the first 256-row CTA-pair boundary, one in the middle and the last pair's
# sequences.  With guidance the same token rows are also head rows R + r, i.e. tiles in the second half.
def test_mar256_full_size_sampled_sequences():
    # The benchmark's launch configuration (B=64, gamma=8, T=100, guidance, bf16-valued weights) on the GPU;
    # 16 sequences per 128-row tile: 15 | 16 straddle a tile, 31 | 32 a pair of tiles.
    _sampled("mar256", [0, 15, 16, 31, 32, 47, 62, 63], "mar256 sampled")


def test_mar256_full_size_rounds_repeat_bit_for_bit():
    # Overlapping launches, the double-buffered condition vector and reused workspace must not make a round depend on
    # what ran before it: the same inputs give the same bits every time, fused and as three calls.
    inp = gen.make_round_inputs(gen.WORKLOADS["mar256"])
    dr, first = _run(inp, fused=True)
    keys = ("x0", "mu1_q", "mu1_p", "logratio", "n_accept", "accept_mask", "x_new", "n_prop", "flags")
    for rep in range(3):
        dr.fused_round() if rep != 1 else dr.three_calls()
        again = dr.results()
        for k in keys:
            np.testing.assert_array_equal(first[k], again[k], err_msg=f"{k} (repeat {rep})")
    dr.ctx.close()


def test_ar_stress_full_size_sampled_sequences():
    # B=256, gamma=16, T=50, no guidance, draft = perturbed target: sequences on both sides of a tile boundary
    _sampled("ar_stress", [0, 7, 8, 15, 16, 128, 254, 255], "ar_stress sampled")


def test_mar512_full_size_sampled_sequences():
    # B=32, gamma=32 (the largest draft length the scan supports), T=100, 12x1536 target head; four sequences per
    # 128-row tile: 3 | 4 straddle a tile, 7 | 8 a pair of tiles
    _sampled("mar512", [0, 3, 4, 7, 8, 16, 30, 31], "mar512 sampled")


def test_large_target_full_size_sampled_sequences():
    # B=128, gamma=16, T=100, guidance: 4096 head rows = 32 row tiles in CTA pairs, W=1536 = 12 column tiles; eight
    # sequences per tile: 7 | 8 straddle a tile, 15 | 16 a pair
    _sampled("large_target", [0, 7, 8, 15, 16, 64, 126, 127], "large_target sampled")


def test_target_only_prefill_rows():
    # Token pre-filling (Sec. 3.2): the first tokens come from the target head alone, i.e. csd_draft_denoise
    # given the target head samples x0 at every step including the last.
    from paper_2411_11925_b200.runner import DeviceRound
    wl = _wl(B=9, gamma=4, T=12, bf16=True, cfg=True, cfg_scale=3.0, draft=gen.HeadSpec(2, 256, 256))
    inp = gen.make_round_inputs(wl)
    dr = DeviceRound(inp)
    x0 = torch.zeros_like(dr.x0); mu1 = torch.zeros_like(dr.x0)
    dr.ctx.csd_draft_denoise(dr.head_p, dr.sched_p, wl.R, wl.cfg, wl.cfg_scale, dr.z_p, dr.x_T, dr.eps, x0, mu1, None)
    dr.ctx.sync()
    sched = orc.ddpm_schedule(inp.beta, wl.tau)
    ref = orc.denoise(orc.make_mlp_head(inp.w_p, inp.z_p, inp.tfeat, wl.cfg, wl.cfg_scale), sched, inp.x_T, inp.eps,
                      sample_last=True)
    assert float(np.max(np.abs(x0.cpu().numpy() - ref["x0"]))) <= 8e-3
    assert float(np.max(np.abs(mu1.cpu().numpy() - ref["mu1"]))) <= 8e-3
    dr.ctx.close()


@pytest.mark.parametrize("op", ["f32", "f16"])
def test_degenerate_sizes_single_row_single_step_widest_scan(op):
    # R = 1 (one sequence, one position), T = 1 (the chain is a single step), and gamma = 32 (every lane of the scan)
    for kw in (dict(B=1, gamma=1, T=1), dict(B=2, gamma=32, T=2), dict(B=1, gamma=3, T=3, cfg=True, cfg_scale=1.5)):
        wl = _wl(bf16=op != "f32", operand=op, draft=gen.HeadSpec(1, 128, 64), target=gen.HeadSpec(1, 128, 128), **kw)
        _check(gen.make_round_inputs(wl), f"degenerate {op} {kw}")


@pytest.mark.parametrize("op", ["bf16", "f16"])
def test_chain_layouts_agree(op):
    # csd_set_chain_mode.  CHAIN_LAYERS_PLAIN runs three kernels per block everywhere.  The default layout folds
    # LayerNorm into the first layer's epilogue from the second block on where its grid rule applies: the same
    # function rounded differently, so it is held to a quarter of a trajectory's tolerance (short chains here: far
    # inside it).  In either layout csd_round returns the bits of the three calls, and a repeat returns the same bits.
    from paper_2411_11925_b200.runner import DeviceRound
    from paper_2411_11925_b200 import api
    cases = (dict(B=5, gamma=7, T=6, cfg=True, cfg_scale=3.0),
             dict(B=23, gamma=7, T=5, cfg=True, cfg_scale=3.0, draft=gen.HeadSpec(1, 256, 128), target=gen.HeadSpec(2, 384, 192)),
             dict(B=37, gamma=8, T=4, cfg=False, cfg_scale=1.0, draft=gen.HeadSpec(2, 768, 128), target=gen.HeadSpec(3, 1024, 128)),
             dict(B=1, gamma=1, T=1, draft=gen.HeadSpec(1, 128, 64), target=gen.HeadSpec(1, 128, 128)),
             dict(B=3, gamma=5, T=3, cfg=True, cfg_scale=2.0, draft=gen.HeadSpec(1, 128, 64), target=gen.HeadSpec(1, 1152, 128)))
    keys = ("x0", "mu1_q", "mu1_p", "x1_q", "logratio", "n_accept", "accept_mask", "x_new", "n_prop", "flags")
    for kw in cases:
        inp = gen.make_round_inputs(_wl(bf16=True, operand=op, **kw))
        dr = DeviceRound(inp)
        dr.three_calls()
        d = dr.results()                      # default layout
        dr.ctx.set_chain_mode(api.Context.CHAIN_LAYERS_PLAIN)
        dr.three_calls()
        a = dr.results()
        dr.three_calls()
        b = dr.results()
        for k in keys:
            np.testing.assert_array_equal(a[k], b[k], err_msg=f"{kw} {k}")
        dr.fused_round()
        c = dr.results()
        for k in keys:
            if k != "x1_q":
                np.testing.assert_array_equal(a[k], c[k], err_msg=f"fused {kw} {k}")
        for k in ("x0", "mu1_q", "mu1_p"):
            assert float(np.max(np.abs(d[k] - a[k]))) <= TOL_X[op] / 4, (kw, k)
        with pytest.raises(api.CsdError):
            dr.ctx.set_chain_mode(7)          # no such layout
        dr.ctx.close()
