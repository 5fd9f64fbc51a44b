"""CPU-side checks: the C-ABI library loads and exports what include/csd.h declares, the binding's
host helpers agree with the float64 checker, the input generators behave."""
import ctypes
import os
import re

import numpy as np
import torch

from oracle import csd_oracle as orc
from paper_2411_11925_b200 import build, inputs as gen

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "csd.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(csd_[a-z_]+)\s*\(", src)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    path = build.build_library()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 12
    missing = [n for n in names if not hasattr(lib, n)]
    assert not missing, missing


def test_binding_covers_the_header():
    from paper_2411_11925_b200 import api
    assert sorted(api.EXPORTS) == _declared()
    # struct layouts mirror the header
    assert [f[0] for f in api._HeadDesc._fields_] == ["C", "W", "L", "Dz", "F", "dtype", "var_out"]
    hdr = open(os.path.join(ROOT, "include", "csd.h")).read()
    block = hdr[hdr.index("typedef struct {\n  const float *Wz"):hdr.index("} csd_head_weights;")]
    assert re.findall(r"\*(\w+)", block) == list(api.WEIGHT_FIELDS)


def test_null_context_calls_return_invalid_arg_without_a_gpu():
    lib = ctypes.CDLL(build.build_library())
    assert lib.csd_sync(None) == -1
    assert lib.csd_destroy(None) == -1
    assert lib.csd_head_destroy(None) == -1
    assert lib.csd_create(None, 0, None) == -1


def test_ddpm_coefficients_match_the_checker_schedule():
    from paper_2411_11925_b200 import api
    for T, tau in ((10, 1.0), (100, 0.9)):
        beta = gen.beta_linear(T)
        c, s = api.ddpm_coefficients(beta, tau), orc.ddpm_schedule(beta, tau)
        for k in ("a", "b", "sigma"):
            np.testing.assert_allclose(c[k], s[k], rtol=1e-7)


def test_log_sigma_term_matches_the_checker_and_rejects_bad_arguments():
    # csd_log_sigma_term (Eq. 7) is a host-only call of the C library: no GPU needed
    from paper_2411_11925_b200 import api
    beta = gen.beta_linear(50)
    cq, cp = api.ddpm_coefficients(beta, 1.0), api.ddpm_coefficients(beta, 0.9)
    tf = torch.zeros(50, 4)

    class _S(api.Schedule):     # the device feature table is irrelevant here
        def __init__(self, c):
            self.sigma = c["sigma"]; self.T = 50

    got = _S(cq).log_sigma_term(_S(cp), 16)
    want = orc.log_sigma_term(cq["sigma"].astype(np.float64), cp["sigma"].astype(np.float64), 16)
    assert abs(got - want) <= 1e-9 * abs(want) and abs(want - 16 * 49 * np.log(1 / 0.9)) < 1e-3
    assert _S(cq).log_sigma_term(_S(cq), 16) == 0.0
    lib = ctypes.CDLL(build.build_library())
    out = ctypes.c_double()
    bad = np.zeros(3, np.float32)
    fp = ctypes.POINTER(ctypes.c_float)
    assert lib.csd_log_sigma_term(3, bad.ctypes.data_as(fp), bad.ctypes.data_as(fp), 16, ctypes.byref(out)) == -1
    assert lib.csd_log_sigma_term(3, None, None, 16, ctypes.byref(out)) == -1
    assert lib.csd_schedule_ddpm(3, None, ctypes.c_double(1.0), None, None, None) == -1
    assert lib.csd_set_wait_limit(None, ctypes.c_int64(5)) == -1 and lib.csd_selftest_wait_timeout(None) == -1


def test_round_to_bf16_matches_torch_and_is_idempotent():
    rng = np.random.default_rng(0)
    a = (rng.standard_normal(10000) * 10.0 ** rng.integers(-6, 3, 10000)).astype(np.float32)
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    got = gen.round_to_bf16(a)
    np.testing.assert_array_equal(got, want)
    np.testing.assert_array_equal(gen.round_to_bf16(got), got)


def test_inputs_are_seeded_shaped_and_in_range():
    wl = gen.WORKLOADS["tiny_fp32"]
    a, b = gen.make_round_inputs(wl), gen.make_round_inputs(wl)
    for k in gen.WEIGHT_NAMES:
        np.testing.assert_array_equal(a.w_p[k], b.w_p[k])
    np.testing.assert_array_equal(a.eps, b.eps)
    assert a.eps.shape == (wl.T, wl.R, 16) and a.z_q.shape == (wl.Rh, 256) and a.u.shape == (1, 4)
    assert np.all((a.u > 0) & (a.u < 1)) and np.all((a.v > 0) & (a.v < 1))
    c = gen.make_round_inputs(wl, seed_offset=7)
    assert not np.array_equal(a.eps, c.eps)
    assert abs(float(np.abs(a.w_p["Wada"]).max()) - np.sqrt(6.0 / (4 * 256))) < 1e-3   # Xavier bound
    assert wl.target.n_params() == sum(v.size for v in a.w_p.values())


def test_workload_table_matches_the_stated_sizes():
    w = gen.WORKLOADS
    assert (w["mar256"].R, w["mar256"].Rh) == (512, 1024)
    assert (w["large_target"].R, w["large_target"].Rh) == (2048, 4096)
    assert (w["mar512"].R, w["mar512"].Rh) == (1024, 2048)
    assert (w["ar_stress"].R, w["ar_stress"].Rh) == (4096, 4096)
    assert abs(w["mar256"].target.flops_per_row_step() / 1e6 - 67.2) < 0.1
    assert abs(w["mar256"].draft.flops_per_row_step() / 1e6 - 35.7) < 0.1
    assert abs(w["mar256"].flops_per_round() / 1e12 - 10.54) < 0.01
    assert abs(w["large_target"].flops_per_round() / 1e12 - 147.4) < 0.1


def test_select_sequences_slices_rows_consistently():
    wl = gen.Workload(**{**gen.WORKLOADS["tiny_fp32"].__dict__, "B": 3, "cfg": True, "cfg_scale": 2.0})
    inp = gen.make_round_inputs(wl)
    sub = gen.select_sequences(inp, [2, 0])
    g = wl.gamma
    np.testing.assert_array_equal(sub.x_T[:g], inp.x_T[2 * g:3 * g])
    np.testing.assert_array_equal(sub.z_p[sub.wl.R:sub.wl.R + g], inp.z_p[wl.R + 2 * g: wl.R + 3 * g])
    np.testing.assert_array_equal(sub.eps[:, g:], inp.eps[:, :g])
    full, part = orc.round_from_inputs(inp), orc.round_from_inputs(sub)
    np.testing.assert_allclose(part["logratio"], full["logratio"][[2, 0]], rtol=1e-9)
    np.testing.assert_allclose(part["x0"][:g], full["x0"][2 * g:3 * g], atol=1e-12)


def test_ddim_coefficients_agree_with_the_checker_and_reject_bad_arguments():
    import numpy as np
    import pytest
    from oracle import csd_oracle as orc
    from paper_2411_11925_b200 import api, inputs as gen
    beta = gen.beta_linear(1000)
    steps = np.linspace(10, 1000, 100).astype(np.int64)
    for eta in (0.2, 1.0):
        got, want = api.ddim_coefficients(beta, steps, eta), orc.ddim_schedule(beta, steps, eta)
        for k in ("a", "b", "sigma"):
            np.testing.assert_allclose(got[k], want[k], rtol=2e-7, atol=1e-9)
        assert np.all(got["sigma"] > 0)
    with pytest.raises(ValueError):
        api.ddim_coefficients(beta, steps, 0.0)
    with pytest.raises(ValueError):
        api.ddim_coefficients(beta, [5, 3], 1.0)
    with pytest.raises(ValueError):
        api.ddim_coefficients(beta, [1, 1001], 1.0)


def test_bench_launches_its_own_ranks_and_counts_decisions(monkeypatch):
    import argparse
    import bench
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    a = argparse.Namespace(gpus=2, master_port=29999)
    cmd = bench.reexec_argv(a, ["--gpus", "2", "--steps", "4"])
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=2" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[-4:] == ["--gpus", "2", "--steps", "4"]
    assert cmd[-5].endswith("bench.py")
    assert bench.reexec_argv(argparse.Namespace(gpus=1, master_port=1), []) is None
    monkeypatch.setenv("WORLD_SIZE", "2")
    assert bench.reexec_argv(a, []) is None          # already a rank: no second launch
    # decision counters, on a round of the checker standing in for the library's outputs
    wl = gen.Workload(**{**gen.WORKLOADS["tiny_fp32"].__dict__, "B": 6, "T": 3, "perturb_std": 1e-4})
    inp = gen.make_round_inputs(wl)
    inp.z_q = inp.z_p
    ref = orc.round_from_inputs(inp)
    res = {k: np.asarray(ref[k]) for k in ("logratio", "n_accept", "n_prop", "flags", "x0")}
    res["cap_hits"] = np.array([ref["cap_hits"]])
    res["accept_mask"] = (ref["accept"].astype(np.int64) << np.arange(wl.gamma)[None, :]).sum(axis=1)
    d = bench.decision_counts(res, inp.u, wl.gamma)
    assert d["decisions"] == 24 and d["resampled"] == int((ref["n_accept"] < wl.gamma).sum())
    assert abs(d["accept_rate"] - ref["accept"].mean()) < 1e-12
    c = bench.checker_counts(res, ref, inp.u, wl, wl.B)
    assert c["accept_mismatch"] == 0 and c["n_prop_mismatch"] == 0 and c["x0_err"] == 0.0
