"""Device-side status words: a bounded wait that runs out, and a non-finite value at a step update.

Neither case faults, traps or hangs anything.  The wait that runs out is a one-thread kernel waiting, with a limit
of 1e5 cycles, on a barrier nobody arrives at; the non-finite value is an fp16 activation beyond 65504 produced by a
head whose first MLP layer is scaled up."""
import time

import numpy as np
import pytest
import torch

from paper_2411_11925_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def _round(op="f16", scale_w1=1.0, **kw):
    from paper_2411_11925_b200.runner import DeviceRound
    base = dict(B=9, gamma=4, T=5, bf16=op != "f32", operand=op, cfg=True, cfg_scale=3.0,
                draft=gen.HeadSpec(2, 256, 128), target=gen.HeadSpec(2, 256, 128))
    base.update(kw)
    wl = gen.Workload(**{**gen.WORKLOADS["tiny_fp32"].__dict__, **base})
    inp = gen.make_round_inputs(wl)
    if scale_w1 != 1.0:
        inp.w_q = dict(inp.w_q); inp.w_q["W1"] = gen.round_to_bf16(inp.w_q["W1"] * np.float32(scale_w1))
    return DeviceRound(inp)


KEYS = ("x0", "mu1_q", "mu1_p", "logratio", "n_accept", "accept_mask", "x_new", "n_prop", "flags")


def test_wait_that_runs_out_returns_timeout_and_the_context_recovers():
    from paper_2411_11925_b200 import api
    dr = _round()
    dr.fused_round()
    before = dr.results()
    dr.ctx.set_wait_limit(100_000)
    t0 = time.perf_counter()
    dr.ctx.selftest_wait_timeout()
    dr.draft()                         # launched while the status word is up: its kernels return at once
    with pytest.raises(api.CsdError) as e:
        dr.ctx.sync()
    assert time.perf_counter() - t0 < 5.0
    assert e.value.code == -6 and "wait self-test" in str(e.value) and "site 1" in str(e.value), str(e.value)
    dr.ctx.sync()                      # reporting cleared the status
    dr.ctx.set_wait_limit(0)           # back to the default limit
    dr.fused_round()
    after = dr.results()
    for k in KEYS:
        np.testing.assert_array_equal(before[k], after[k], err_msg=k)
    dr.ctx.close()


def test_fp16_activation_overflow_is_reported_as_nonfinite_and_bf16_operands_take_the_same_head():
    from paper_2411_11925_b200 import api
    dr = _round("f16", scale_w1=1.0e5)     # weights up to 1e4 (finite in fp16), activations beyond 65504
    dr.draft()
    with pytest.raises(api.CsdError) as e:
        dr.ctx.sync()
    assert e.value.code == -7 and "65504" in str(e.value), str(e.value)
    dr.ctx.sync()                          # cleared; nothing faulted: the context goes on working
    dr.verify()
    dr.ctx.sync()
    dr.ctx.close()
    ok = _round("bf16", scale_w1=1.0e5)    # fp32 exponent range: the same head runs
    ok.draft()
    ok.ctx.sync()
    assert torch.isfinite(ok.x0).all()
    ok.ctx.close()


def test_contexts_keep_the_callers_current_device():
    from paper_2411_11925_b200 import api
    cur = torch.cuda.current_device()
    ctx = api.Context(0)
    assert torch.cuda.current_device() == cur
    ctx.sync()
    ctx.close()
    assert torch.cuda.current_device() == cur
