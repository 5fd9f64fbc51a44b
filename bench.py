#!/usr/bin/env python
"""Benchmark of the continuous-speculative-decoding hot path: draft tokens/s through
denoise + verify + resample (one step = one speculative round over one synthetic batch).

    python bench.py --gpus N --steps K --warmup W [--workload mar256] [--impl reference]

N > 1 is launched by torch.distributed.run (one rank per GPU).  The path shards by sequence with
replicated heads and no data-path collective (weak scaling: every rank runs its own batch); the
ranks only meet in a barrier and a max-reduction of the measured time.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

# dram__bytes_read + dram__bytes_write per launch of a kernel class, from the ncu capture summarised in
# profiles/mar256_gemm_tc_kernels_ncu_full.md (set to None when the kernel changes after the capture)
NCU_DRAM_BYTES_PER_LAUNCH = {("mar256", "mlp2_gate_residual"): 14.73e6, ("mar256", "adaln_modulate"): 10.67e6,
                             ("mar256", "mlp1_silu"): 10.67e6}

METRIC = "draft tokens/s through denoise+verify+resample"
UNIT = "tokens/s"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mar256")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-profile", action="store_true")
    ap.add_argument("--no-seq", action="store_true", help="skip the sequential-draft variant")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    return ap.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"tflops_sustained": float(p["bf16_tflops_sustained"]), "tflops_burst": float(p["bf16_tflops"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"tflops_sustained": 1400.0, "tflops_burst": 1590.0, "hbm_gbs": 6650.0, "source": "fallback"}


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Reads (never sets) SM clock and throttle reasons every 100 ms while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz, self._stop = [], set(), None, threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20,
                 "hw_thermal_slowdown": 0x40, "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.1)

    def start(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self) -> dict:
        self._stop.set()
        if self._thr is not None:
            self._thr.join(timeout=2)
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ----------------------------------------------------------------------------- CPU checker leg
def time_oracle(wl_name: str, seconds_hint: float = 15.0, repeats: int = 1):
    """Times the float64 checker, as it stands, on a bounded sample of the workload: whole
    sequences (all gamma positions, both guidance halves, all T steps, both heads + verify +
    resample).  Returns (tokens/s, threads, description, seconds per repeat list)."""
    from oracle import csd_oracle as orc
    from paper_2411_11925_b200 import inputs as gen
    wl = gen.WORKLOADS[wl_name]
    flops_seq = wl.flops_per_round() / wl.B
    nseq = max(1, min(wl.B, int(seconds_hint * 40e9 / flops_seq)))       # ~40 GFLOP/s fp64 guess
    inp = gen.make_round_inputs(wl)
    sub = gen.select_sequences(inp, range(nseq))
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        orc.round_from_inputs(sub)
        times.append(time.perf_counter() - t0)
    tok = nseq * wl.gamma
    desc = (f"{nseq} of {wl.B} sequences of {wl_name} ({tok} draft tokens: all {wl.gamma} positions, "
            f"{'both guidance halves, ' if wl.cfg else ''}T={wl.T}, draft+target heads, verify, resample), float64 numpy")
    return tok / float(np.mean(times)), threads, desc, times


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2411_11925_b200 import inputs as gen
    wl = gen.WORKLOADS[args.workload]
    # each "step" is one bounded sample; keep the whole run to a few minutes
    per_step = max(2.0, min(15.0, 150.0 / max(1, args.steps + args.warmup)))
    val, threads, desc, times = time_oracle(args.workload, per_step, repeats=args.steps + args.warmup)
    times = times[args.warmup:] if len(times) > args.warmup else times
    tok = int(desc.split("(")[1].split(" ")[0])
    val = tok / float(np.mean(times))
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(times)),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "B": wl.B, "gamma": wl.gamma, "T": wl.T, "cfg_scale": wl.cfg_scale,
                       "sample": desc},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2411_11925_b200 import inputs as gen
    from paper_2411_11925_b200.runner import DeviceRound

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    wl = gen.WORKLOADS[args.workload]
    peaks = load_peaks()

    # several independent input sets (fresh z, noise, uniforms per round), shared heads; rank-dependent seed
    nsets = 3
    stream = torch.cuda.Stream(device=dev)
    from paper_2411_11925_b200 import api
    ctx = api.Context(local, stream)
    inp0 = gen.make_round_inputs(wl, seed_offset=1000 * rank)
    rounds = [DeviceRound(inp0, ctx=ctx, device=local)]
    for i in range(1, nsets):
        inp = gen.make_round_inputs(wl, seed_offset=1000 * rank + 17 * i, weights=False)
        inp.w_q, inp.w_p = inp0.w_q, inp0.w_p
        rounds.append(DeviceRound(inp, ctx=ctx, device=local, heads=(rounds[0].head_q, rounds[0].head_p)))
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)     # > 126 MB L2

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn_of_step, steps, sampler=None):
        """Each step timed by its own CUDA-event pair on the library's stream; an L2 flush (not timed)
        runs between steps.  Returns total seconds of the `steps` steps."""
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        if sampler:
            sampler.start()
        with torch.cuda.stream(stream):
            for i in range(steps):
                flush.fill_(i & 0xFF)
                evs[i][0].record(stream)
                fn_of_step(i)
                evs[i][1].record(stream)
        barrier()
        return sum(a.elapsed_time(b) for a, b in evs) * 1e-3

    dev_step = lambda i: rounds[i % nsets].fused_round()
    # warm-up (also grows the workspaces)
    timed(dev_step, args.warmup)
    ctx.sync()
    sampler = ClockSampler(local)
    l0 = ctx.launch_count()
    secs = timed(dev_step, args.steps, sampler)
    launches = ctx.launch_count() - l0
    clocks = sampler.stop()
    ctx.sync()

    # end to end: host buffers in, host buffers out, copies inside the timed region
    hosts = [r.make_host_buffers() for r in rounds]
    host_step = lambda i: rounds[i % nsets].host_round(hosts[i % nsets])
    if args.no_e2e:
        e2e_secs = float("nan")
    else:
        timed(host_step, 1)
        e2e_secs = timed(host_step, args.steps)
    in_names = ("z_q", "z_p", "x_T", "eps", "u", "xi", "v")
    out_names = ("x0", "mu1_q", "mu1_p", "logratio", "n_accept", "accept_mask", "x_new", "n_prop", "flags", "cap_hits")
    h2d = sum(hosts[0][n].numel() * hosts[0][n].element_size() for n in in_names)
    d2h = sum(hosts[0][n].numel() * hosts[0][n].element_size() for n in out_names)

    # Sequential-draft variant: how an autoregressive loop has to call the draft head, one position at a time
    # (gamma calls of csd_draft_denoise with B tokens = B (1 + cfg) head rows each).  Few rows per call: the
    # binding resource is streaming the draft head's weights once per denoising step.
    seq = None
    if world == 1 and not args.no_seq:
        wl1 = gen.Workload(**{**wl.__dict__, "gamma": 1})
        inp1 = gen.make_round_inputs(wl1, seed_offset=5000, weights=False)
        inp1.w_q, inp1.w_p = inp0.w_q, inp0.w_p
        r1 = DeviceRound(inp1, ctx=ctx, device=local, heads=(rounds[0].head_q, rounds[0].head_p))
        seq_step = lambda i: [r1.draft() for _ in range(wl.gamma)]
        timed(seq_step, 2)
        seq_steps = max(2, min(args.steps, 5))
        seq_secs = timed(seq_step, seq_steps)
        d = wl.draft
        wbytes = 2.0 * (d.W * d.Dz + d.L * 5 * d.W * d.W + 2 * d.W * d.W)     # 16-bit GEMM weights of the draft head
        per_call = seq_secs / (seq_steps * wl.gamma)
        seq = {"calls_per_round": wl.gamma, "head_rows_per_call": wl.B * (2 if wl.cfg else 1),
               "ms_per_call": 1e3 * per_call, "value": wl.B * wl.gamma * seq_steps / seq_secs, "unit": UNIT,
               "bound": "hbm", "weight_bytes_per_step": wbytes,
               "achieved": wbytes * wl.T / per_call / 1e9, "peak": peaks["hbm_gbs"], "roofline_unit": "GB/s",
               "frac": wbytes * wl.T / per_call / 1e9 / peaks["hbm_gbs"],
               "note": "algorithmic bytes = draft weight bytes x T per call; the weights fit L2 (126 MB), so the "
                       "fraction says how far the call is from streaming them from HBM once per step"}

    # Token pre-filling (Sec. 3.2): the first tokens of an image come from the target head alone, one
    # csd_draft_denoise call with the target head over B * prefill tokens; timed separately.
    prefill = None
    if world == 1 and wl.prefill and wl.prefill == wl.gamma and not args.no_seq:
        r0 = rounds[0]
        px0, pmu = torch.zeros_like(r0.x0), torch.zeros_like(r0.x0)
        pre_step = lambda i: ctx.csd_draft_denoise(r0.head_p, r0.sched_p, wl.R, wl.cfg, wl.cfg_scale, r0.z_p, r0.x_T, r0.eps,
                                                   px0, pmu, None)
        timed(pre_step, 1)
        pre_steps = max(2, min(args.steps, 5))
        pre_secs = timed(pre_step, pre_steps)
        t = wl.target
        fl = (2 if wl.cfg else 1) * wl.R * wl.T * 2.0 * (2 * t.C * t.W + 5 * t.L * t.W * t.W + 2 * t.W * t.W)
        prefill = {"tokens": wl.R, "ms": 1e3 * pre_secs / pre_steps, "value": wl.R * pre_steps / pre_secs, "unit": "prefilled tokens/s",
                   "algorithmic_tflops": fl * pre_steps / pre_secs / 1e12,
                   "frac_of_tensor_peak": fl * pre_steps / pre_secs / 1e12 / peaks["tflops_sustained"]}

    # Exact single-path criterion (Eq. 2): the target scores the draft's recorded trajectory.  Its T evaluations are
    # independent rows, so the call is throughput-bound: reported against the tensor roofline with algorithmic
    # FLOPs = (1 + cfg) R T F_target.
    single = None
    if world == 1 and not args.no_seq:
        r0 = rounds[0]
        r0.draft_traj()
        sp_step = lambda i: r0.verify_single_path()
        timed(sp_step, 2)
        l1 = ctx.launch_count()
        sp_steps = max(2, min(args.steps, 5))
        sp_secs = timed(sp_step, sp_steps)
        t = wl.target
        fl = (2 if wl.cfg else 1) * wl.R * wl.T * 2.0 * (2 * t.C * t.W + 5 * t.L * t.W * t.W + 2 * t.W * t.W)
        single = {"call": "csd_verify_single_path", "ms": 1e3 * sp_secs / sp_steps, "value": wl.R * sp_steps / sp_secs,
                  "unit": "verified tokens/s", "launches_per_call": int((ctx.launch_count() - l1) // sp_steps),
                  "bound": "tensor", "achieved": fl * sp_steps / sp_secs / 1e12, "peak": peaks["tflops_sustained"],
                  "roofline_unit": "TFLOP/s", "frac": fl * sp_steps / sp_secs / 1e12 / peaks["tflops_sustained"]}

    # per-kernel-class device time over the same steps (events around every launch: separate pass)
    prof = None
    if not args.no_profile:
        ctx.profile(True)
        # the three calls one after the other: the same kernels and grids as csd_round, but the draft and the
        # target chain do not share the GPU, so a launch's duration is the kernel's own
        timed(lambda i: rounds[i % nsets].three_calls(), min(args.steps, 3))
        prof = ctx.profile_read()
        ctx.profile(False)

    if world > 1:
        t = torch.tensor([secs, e2e_secs], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        secs, e2e_secs = float(t[0]), float(t[1])
    tokens = wl.R * args.steps * world
    value = tokens / secs

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None,
                "dtype": {"f16": "f16 (bf16-valued weights, fp32 accumulate)", "bf16": "bf16", "f32": "f32"}[wl.operand_format],
                "data": "synthetic",
                "config": {"workload": wl.name, "B_per_gpu": wl.B, "gamma": wl.gamma, "T": wl.T, "cfg_scale": wl.cfg_scale,
                           "draft_head": f"{wl.draft.L}x{wl.draft.W} (z {wl.draft.Dz})",
                           "target_head": f"{wl.target.L}x{wl.target.W} (z {wl.target.Dz})",
                           "parallelism": f"sequences sharded over {world} GPU(s), heads replicated, no collective",
                           "l2": "256 MB L2 flush between timed steps (outside the per-step event pairs)",
                           "call": "csd_round"},
                "clocks": clocks,
                "e2e": {"value": tokens / e2e_secs, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                        "d2h_bytes_per_step": int(d2h), "call": "csd_round_host (pinned host buffers)"},
                "gpu_launches": int(launches)}
        algo_flops = wl.flops_per_round()
        line["algorithmic_tflops"] = algo_flops * args.steps * world / secs / 1e12 / world
        line["path_frac_of_tensor_peak"] = line["algorithmic_tflops"] / peaks["tflops_sustained"]
        if prof:
            gemm = {k: v for k, v in prof.items() if k != "step" and v["launches"] > 0}
            top = max(gemm, key=lambda k: gemm[k]["ms"])
            tot_ms = sum(v["ms"] for v in prof.values())
            ach = gemm[top]["flops"] / (gemm[top]["ms"] * 1e-3) / 1e12
            line["roofline"] = {"bound": "tensor", "kernel": top, "achieved": ach, "peak": peaks["tflops_sustained"],
                                "unit": "TFLOP/s", "frac": ach / peaks["tflops_sustained"],
                                "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get((wl.name, top)),
                                "peak_source": f"{peaks['source']} bf16 sustained (fp16 has the same nominal rate)",
                                "avg_launch_us": 1e3 * gemm[top]["ms"] / gemm[top]["launches"],
                                "per_class": {k: {"launches": v["launches"], "ms": round(v["ms"], 3),
                                                  "share": round(v["ms"] / tot_ms, 4),
                                                  "tflops": (v["flops"] / (v["ms"] * 1e-3) / 1e12 if v["ms"] > 0 else 0.0)}
                                              for k, v in prof.items()}}
        if seq:
            line["sequential_draft"] = seq
        if prefill:
            line["prefill"] = prefill
        if single:
            line["single_path"] = single
        if not args.no_cpu_baseline and world == 1:
            val, threads, desc, _ = time_oracle(args.workload, 15.0)
            line["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
