"""The comparator used by the GPU parity tests must reject a wrong log-ratio or decision (CPU only).

A stand-in for the library's output is built from the float64 checker's own round (means perturbed by a
trajectory-sized error, everything downstream recomputed consistently); the comparator must accept it.  Mistakes
are then planted on that CPU copy: a log-ratio computed from a mean that is 1e-3 off, a flipped decision away from
the band, a wrong prefix length, a wrong proposal count."""
import copy

import numpy as np
import pytest

from oracle import csd_oracle as orc
from paper_2411_11925_b200 import inputs as gen

from _parity import compare_round, eq8_float64


def _case(op="f16", seed=3):
    wl = gen.Workload(**{**gen.WORKLOADS["tiny_fp32"].__dict__, "B": 24, "gamma": 6, "T": 4, "perturb_std": 1e-4,
                         "bf16": op != "f32", "operand": op,
                         "draft": gen.HeadSpec(1, 128, 64), "target": gen.HeadSpec(1, 128, 64)})
    inp = gen.make_round_inputs(wl)
    inp.z_q = inp.z_p
    sq = orc.ddpm_schedule(inp.beta, wl.tau)
    eq = orc.make_mlp_head(inp.w_q, inp.z_q, inp.tfeat, wl.cfg, wl.cfg_scale)
    ep = orc.make_mlp_head(inp.w_p, inp.z_p, inp.tfeat, wl.cfg, wl.cfg_scale)
    ref = orc.csd_round(eq, ep, sq, sq, inp.x_T, inp.eps, inp.u, inp.xi, inp.v, wl.B, wl.gamma, wl.cap)
    s1 = float(sq["sigma"][0])
    # consistent stand-in: means off by a small error, x0 follows mu1_q, ratio / scan / resampling recomputed from them
    rng = np.random.default_rng(seed)
    err = 2e-5 if op != "f32" else 2e-7
    g = {"mu1_q": (ref["mu1_q"] + err * rng.standard_normal(ref["mu1_q"].shape)).astype(np.float32),
         "mu1_p": (ref["mu1_p"] + err * rng.standard_normal(ref["mu1_p"].shape)).astype(np.float32)}
    g["x0"] = (g["mu1_q"].astype(np.float64) + s1 * inp.eps[0]).astype(np.float32)
    lr, _, _ = eq8_float64(g["x0"], g["mu1_q"], g["mu1_p"], s1, s1, 0.0)
    g["logratio"] = lr.reshape(wl.B, wl.gamma).astype(np.float32)
    n, acc = orc.accept_prefix(g["logratio"].astype(np.float64), inp.u)
    g["n_accept"] = n
    g["accept_mask"] = (acc.astype(np.int64) << np.arange(wl.gamma)[None, :]).sum(axis=1).astype(np.int32)
    rs = orc.resample(n, g["mu1_p"].astype(np.float64), g["mu1_q"].astype(np.float64), s1, s1, 0.0, inp.xi, inp.v,
                      wl.gamma, wl.cap)
    g["x_new"], g["n_prop"], g["flags"] = rs["x_new"].astype(np.float32), rs["n_prop"], rs["flags"]
    g["cap_hits"] = np.array([rs["cap_hits"]], dtype=np.int32)
    return wl, inp, ref, g, s1


def _cmp(wl, inp, ref, g, s1):
    return compare_round(g, ref, wl, s1, s1, inp.u, inp.v, "harness", xi=inp.xi)


@pytest.mark.parametrize("op", ["f32", "f16"])
def test_consistent_stand_in_passes(op):
    wl, inp, ref, g, s1 = _case(op)
    st = _cmp(wl, inp, ref, g, s1)
    assert st["decisions"] == wl.B * wl.gamma and 0.02 < st["accept_rate"] < 0.999


def test_logratio_from_a_mean_that_is_off_by_1e_3_is_rejected():
    wl, inp, ref, g, s1 = _case()
    bad = copy.deepcopy(g)
    lr, _, _ = eq8_float64(g["x0"], g["mu1_q"], g["mu1_p"] + np.float32(1e-3), s1, s1, 0.0)
    bad["logratio"] = lr.reshape(wl.B, wl.gamma).astype(np.float32)
    with pytest.raises(AssertionError):
        _cmp(wl, inp, ref, bad, s1)


def test_dropped_sigma_term_is_rejected():
    # a ratio kernel that forgot log Sigma: the checker's round has log Sigma != 0 when the schedules differ
    wl, inp, ref, g, s1 = _case()
    ref2 = dict(ref); ref2["log_sigma"] = 0.7; ref2["logratio"] = ref["logratio"] + 0.7
    with pytest.raises(AssertionError):
        _cmp(wl, inp, ref2, g, s1)


def test_flipped_decision_outside_the_band_is_rejected():
    wl, inp, ref, g, s1 = _case()
    margin = np.abs(ref["logratio"] - np.log(inp.u.astype(np.float64)))
    b, i = np.unravel_index(np.argmax(margin), margin.shape)
    bad = copy.deepcopy(g)
    bad["accept_mask"][b] ^= np.int32(1 << i)
    with pytest.raises(AssertionError):
        _cmp(wl, inp, ref, bad, s1)


def test_wrong_prefix_length_is_rejected():
    wl, inp, ref, g, s1 = _case()
    bad = copy.deepcopy(g)
    b = int(np.argmax(g["n_accept"] > 0))
    bad["n_accept"][b] -= 1
    with pytest.raises(AssertionError):
        _cmp(wl, inp, ref, bad, s1)


def test_wrong_proposal_count_is_rejected():
    wl, inp, ref, g, s1 = _case()
    bad = copy.deepcopy(g)
    rows = np.flatnonzero(g["n_prop"] > 0)
    assert rows.size
    # one more proposal than the checker consumed, although v was far below the threshold of the accepted one
    far = [b for b in rows if g["n_prop"][b] < wl.cap]
    bad["n_prop"][far[0]] += 1
    with pytest.raises(AssertionError):
        _cmp(wl, inp, ref, bad, s1)
