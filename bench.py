#!/usr/bin/env python
"""Benchmark of the continuous-speculative-decoding hot path: draft tokens/s through
denoise + verify + resample (one step = one speculative round over one synthetic batch).

    python bench.py --gpus N --steps K --warmup W [--workload mar256] [--impl reference]

N > 1 runs one rank per GPU under torch.distributed.run (started by the caller, or by this file itself when it is
run plainly with --gpus N).  The path shards by sequence with
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

# dram__bytes_read + dram__bytes_write per launch of a kernel class, from the ncu capture summarised under
# profiles/ for (workload, class); absent = no capture of the kernel as it stands (reported as null)
NCU_DRAM_BYTES_PER_LAUNCH = {
    # profiles/mar256_sequential_draft_sb_chain_kernel_ncu.md: 99.4 MB read + 51.8 MB written per launch
    ("mar256", "sb_chain"): 151.2e6,
    # profiles/mar256_persistent_chain_kernel_ncu.md: 6.02 GB read + 43.6 MB written per launch of the target chain
    ("mar256", "pchain_target"): 6.062e9,
}

# Sequences of each workload that the float64 checker evaluates when it is timed (the first n of the batch): the
# CPU-baseline leg and the reference arm time the very same sample.
SAMPLE_SEQS = {"tiny_fp32": 1, "mar256": 4, "large_target": 1, "mar512": 1, "ar_stress": 4}

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
    ap.add_argument("--no-seq", action="store_true", help="skip the sequential-draft, prefill and single-path legs")
    ap.add_argument("--no-workloads", action="store_true", help="skip the short runs of the other workloads")
    ap.add_argument("--rounds-per-step", type=int, default=0,
                    help="speculative rounds per timed step (0: one image-shaped pass = tokens / gamma rounds)")
    ap.add_argument("--master-port", type=int, default=29533)
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


def reexec_argv(args, argv):
    """Command line that runs this file as `args.gpus` ranks under torch.distributed.run on this node, or None when
    the process already is a rank (WORLD_SIZE set) or one GPU is asked for."""
    if args.gpus <= 1 or "WORLD_SIZE" in os.environ:
        return None
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(args.master_port), os.path.abspath(__file__)] + list(argv)


# ----------------------------------------------------------------------------- CPU checker leg
def oracle_sample(wl_name: str):
    """The bounded sample the checker is timed on: the first SAMPLE_SEQS[wl] whole sequences of the workload's
    round (seed offset 0: the inputs rank 0's first device round uses)."""
    from paper_2411_11925_b200 import inputs as gen
    wl = gen.WORKLOADS[wl_name]
    nseq = min(wl.B, SAMPLE_SEQS.get(wl_name, 1))
    inp = gen.make_round_inputs(wl)
    sub = gen.select_sequences(inp, range(nseq))
    tok = nseq * wl.gamma
    desc = (f"{nseq} of {wl.B} sequences of {wl_name} ({tok} draft tokens: all {wl.gamma} positions, "
            f"{'both guidance halves, ' if wl.cfg else ''}T={wl.T}, draft+target heads, verify, resample), float64 numpy")
    return sub, tok, desc


def oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def time_oracle(wl_name: str, repeats: int = 0, budget_s: float = 15.0):
    """Times the float64 checker, as it stands, on oracle_sample().  repeats = 0: as many runs as fit about
    `budget_s` seconds (at least one, at most eight).  Returns (tokens/s, threads, description, seconds per run,
    the checker's result of the sample)."""
    from oracle import csd_oracle as orc
    sub, tok, desc = oracle_sample(wl_name)
    times, res = [], None
    n = repeats if repeats > 0 else 1
    i = 0
    while i < n:
        t0 = time.perf_counter()
        res = orc.round_from_inputs(sub)
        times.append(time.perf_counter() - t0)
        i += 1
        if repeats <= 0 and i == 1:
            n = int(max(1, min(8, round(budget_s / max(times[0], 1e-3)))))
    return tok / float(np.mean(times)), oracle_threads(), desc, times, res


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2411_11925_b200 import inputs as gen
    wl = gen.WORKLOADS[args.workload]
    # each "step" is one run of the bounded sample
    _, threads, desc, times, _ = time_oracle(args.workload, repeats=args.steps + args.warmup)
    times = times[args.warmup:] if len(times) > args.warmup else times
    tok = min(wl.B, SAMPLE_SEQS.get(args.workload, 1)) * wl.gamma
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
def decision_counts(res: dict, u: np.ndarray, gamma: int) -> dict:
    """What the accept test and the resampler did in one round, from the library's own outputs: decisions whose margin
    |logR - log u| lies inside the 5e-2 log-ratio tolerance band (the only ones a tolerance-sized error could flip),
    accepted-prefix statistics, resampling proposals and cap hits."""
    lr = res["logratio"].astype(np.float64)
    margin = np.abs(lr - np.log(u.astype(np.float64)))
    resampled = (res["flags"] & 1) != 0
    return {"decisions": int(lr.size), "band_count": int((margin <= 5e-2).sum()),
            "accept_rate": float((np.log(u.astype(np.float64)) <= lr).mean()),
            "mean_n_accept": float(res["n_accept"].mean()), "all_accepted": int((res["n_accept"] == gamma).sum()),
            "resampled": int(resampled.sum()),
            "mean_n_prop": float(res["n_prop"][resampled].mean()) if resampled.any() else 0.0,
            "cap_hits": int(res["cap_hits"][0])}


def checker_counts(gpu: dict, ref: dict, u: np.ndarray, wl, nseq: int) -> dict:
    """The library's first device round against the checker's result on the timed sample (its first nseq sequences)."""
    rows = nseq * wl.gamma
    g_lr, r_lr = gpu["logratio"][:nseq].astype(np.float64), ref["logratio"]
    logu = np.log(u[:nseq].astype(np.float64))
    gm = gpu["accept_mask"][:nseq].astype(np.int64) & 0xFFFFFFFF
    acc_g = ((gm[:, None] >> np.arange(wl.gamma)[None, :]) & 1).astype(bool)
    acc_r = logu <= r_lr
    same = np.all(acc_g == acc_r, axis=1)
    res = same & (ref["n_accept"] < wl.gamma)
    return {"sequences": nseq, "decisions": int(acc_r.size),
            "x0_err": float(np.max(np.abs(gpu["x0"][:rows] - ref["x0"]))),
            "logr_err": float(np.max(np.abs(g_lr - r_lr))),
            "band_count": int((np.abs(r_lr - logu) <= 5e-2).sum()),
            "accept_mismatch": int((acc_g != acc_r).sum()),
            "n_accept_mismatch": int((gpu["n_accept"][:nseq] != ref["n_accept"]).sum()),
            "n_prop_mismatch": int((gpu["n_prop"][:nseq][res] != ref["n_prop"][res]).sum()),
            "cap_hits_checker": int(ref["cap_hits"])}


def head_flops(h, rows_steps: float) -> float:
    return rows_steps * 2.0 * (2 * h.C * h.W + 5 * h.L * h.W * h.W + 2 * h.W * h.W)


def measure(name, args, peaks, steps, warmup, rounds_per_step, full):
    """All timings of one workload on this rank's GPU.  A step = rounds_per_step speculative rounds (csd_round) on
    rotating input sets; steps are timed by their own CUDA-event pairs on the library's stream with an L2 flush (not
    timed) between them.  full: also the host-buffer leg, the per-class profile and the checker comparison."""
    import torch
    import torch.distributed as dist
    from paper_2411_11925_b200 import api, inputs as gen
    from paper_2411_11925_b200.runner import DeviceRound

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dev = torch.device("cuda", local)
    wl = gen.WORKLOADS[name]
    nsets = 3
    stream = torch.cuda.Stream(device=dev)
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

    def timed(fn_of_step, nsteps, sampler=None):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(nsteps)]
        barrier()
        if sampler:
            sampler.start()
        with torch.cuda.stream(stream):
            for i in range(nsteps):
                flush.fill_(i & 0xFF)
                evs[i][0].record(stream)
                fn_of_step(i)
                evs[i][1].record(stream)
        barrier()
        return sum(a.elapsed_time(b) for a, b in evs) * 1e-3

    rps = rounds_per_step

    def dev_step(i):
        for j in range(rps):
            rounds[(i * rps + j) % nsets].fused_round()

    timed(dev_step, warmup)
    ctx.sync()
    sampler = ClockSampler(local)
    l0 = ctx.launch_count()
    secs = timed(dev_step, steps, sampler)
    launches = ctx.launch_count() - l0
    clocks = sampler.stop()
    ctx.sync()
    out = {"wl": wl, "secs": secs, "launches": int(launches), "clocks": clocks, "rounds": steps * rps}
    # decisions of one round on rank 0's first input set (deterministic: the same bits every round)
    rounds[0].fused_round()
    res0 = rounds[0].results()
    out["res0"], out["inp0"] = res0, inp0
    out["decisions"] = decision_counts(res0, inp0.u, wl.gamma)

    if full and not args.no_e2e:
        hosts = [r.make_host_buffers() for r in rounds]

        def host_step(i):
            for j in range(rps):
                k = (i * rps + j) % nsets
                rounds[k].host_round(hosts[k])
        timed(host_step, 1)
        out["e2e_secs"] = timed(host_step, steps)
        in_names = ("z_q", "z_p", "x_T", "eps", "u", "xi", "v")
        out_names = ("x0", "mu1_q", "mu1_p", "logratio", "n_accept", "accept_mask", "x_new", "n_prop", "flags", "cap_hits")
        out["h2d"] = rps * sum(hosts[0][n].numel() * hosts[0][n].element_size() for n in in_names)
        out["d2h"] = rps * sum(hosts[0][n].numel() * hosts[0][n].element_size() for n in out_names)
    else:
        out["e2e_secs"] = float("nan")

    few = max(3, min(steps, 5))
    # The two chains of a round on their own (csd_draft_denoise, csd_verify): with the persistent chain kernel a call
    # is one launch, so this is the kernel's duration; and the same round from the layer kernels only.
    if full:
        l1 = ctx.launch_count()
        timed(lambda i: rounds[i % nsets].draft(), 2)
        d_launches = (ctx.launch_count() - l1) // 2
        d_secs = timed(lambda i: rounds[i % nsets].draft(), few)
        timed(lambda i: rounds[i % nsets].verify(), 2)
        v_secs = timed(lambda i: rounds[i % nsets].verify(), few)
        ctx.set_chain_mode(api.Context.CHAIN_LAYER_KERNELS)
        timed(lambda i: rounds[i % nsets].fused_round(), 3)
        lk_secs = timed(lambda i: rounds[i % nsets].fused_round(), few)
        ctx.set_chain_mode(api.Context.CHAIN_LAYERS)
        out["chains"] = {"draft_ms": 1e3 * d_secs / few, "verify_ms": 1e3 * v_secs / few,
                         "draft_launches_per_call": int(d_launches),
                         "persistent_chain_kernel": bool(d_launches < 50),
                         "layer_kernels_ms_per_round": 1e3 * lk_secs / few}

    # Sequential-draft variant: how an autoregressive loop has to call the draft head, one position at a time
    # (gamma calls of csd_draft_denoise with B tokens = B (1 + cfg) head rows each).  Few rows per call: the
    # binding resource is streaming the draft head's weights once per denoising step.
    if full and world == 1 and not args.no_seq:
        wl1 = gen.Workload(**{**wl.__dict__, "gamma": 1})
        inp1 = gen.make_round_inputs(wl1, seed_offset=5000, weights=False)
        inp1.w_q, inp1.w_p = inp0.w_q, inp0.w_p
        r1 = DeviceRound(inp1, ctx=ctx, device=local, heads=(rounds[0].head_q, rounds[0].head_p))
        seq_step = lambda i: [r1.draft() for _ in range(wl.gamma)]
        timed(seq_step, 3)
        layers_secs = timed(seq_step, few)
        # the persistent small-batch kernel (csd_set_chain_mode): chains of at most 128 head rows
        ctx.set_chain_mode(api.Context.CHAIN_SMALL_BATCH)
        timed(seq_step, 3)
        l1 = ctx.launch_count()
        seq_secs = timed(seq_step, few)
        launches_per_call = int((ctx.launch_count() - l1) // (few * wl.gamma))
        ctx.set_chain_mode(api.Context.CHAIN_LAYERS)
        d = wl.draft
        wbytes = 2.0 * (d.W * d.Dz + d.L * 5 * d.W * d.W + 2 * d.W * d.W)     # 16-bit GEMM weights of the draft head
        per_call = seq_secs / (few * wl.gamma)
        out["sequential_draft"] = {
            "calls_per_round": wl.gamma, "head_rows_per_call": wl.B * (2 if wl.cfg else 1),
            "chain_mode": "CSD_CHAIN_SMALL_BATCH" if launches_per_call < 50 else "CSD_CHAIN_LAYERS (small-batch kernel not eligible)",
            "ms_per_call": 1e3 * per_call, "us_per_denoising_step": 1e6 * per_call / wl.T,
            "layer_kernels_ms_per_call": 1e3 * layers_secs / (few * wl.gamma),
            "launches_per_call": launches_per_call,
            "value": wl.B * wl.gamma * few / seq_secs, "unit": UNIT,
            "bound": "hbm", "weight_bytes_per_step": wbytes, "achieved": wbytes * wl.T / per_call / 1e9,
            "peak": peaks["hbm_gbs"], "roofline_unit": "GB/s", "frac": wbytes * wl.T / per_call / 1e9 / peaks["hbm_gbs"],
            "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get((wl.name, "sb_chain")) if launches_per_call < 50 else None,
            "note": "algorithmic bytes = draft weight bytes x T per call; the weights fit L2 (126 MB), so the "
                    "fraction says how far the call is from streaming them from HBM once per step"}

    # Token pre-filling (Sec. 3.2): the first tokens of an image come from the target head alone, one
    # csd_draft_denoise call with the target head over B * prefill tokens; timed separately.
    if world == 1 and wl.prefill and wl.prefill == wl.gamma and not args.no_seq:
        r0 = rounds[0]
        px0, pmu = torch.zeros_like(r0.x0), torch.zeros_like(r0.x0)
        pre_step = lambda i: ctx.csd_draft_denoise(r0.head_p, r0.sched_p, wl.R, wl.cfg, wl.cfg_scale, r0.z_p, r0.x_T,
                                                   r0.eps, px0, pmu, None)
        timed(pre_step, 3)
        pre_secs = timed(pre_step, few)
        fl = head_flops(wl.target, (2 if wl.cfg else 1) * wl.R * wl.T)
        out["prefill"] = {"tokens": wl.R, "ms": 1e3 * pre_secs / few, "value": wl.R * few / pre_secs,
                          "unit": "prefilled tokens/s", "algorithmic_tflops": fl * few / pre_secs / 1e12,
                          "frac_of_tensor_peak": fl * few / pre_secs / 1e12 / peaks["tflops_sustained"]}

    # Exact single-path criterion (Eq. 2): the target scores the draft's recorded trajectory.  Its T evaluations are
    # independent rows, so the call is throughput-bound: reported against the tensor roofline with algorithmic
    # FLOPs = (1 + cfg) R T F_target.
    if world == 1 and not args.no_seq and wl.operand_format != "f32":
        r0 = rounds[0]
        r0.draft_traj()
        sp_step = lambda i: r0.verify_single_path()
        timed(sp_step, 3)
        l1 = ctx.launch_count()
        sp_secs = timed(sp_step, few)
        fl = head_flops(wl.target, (2 if wl.cfg else 1) * wl.R * wl.T)
        out["single_path"] = {"call": "csd_verify_single_path", "ms": 1e3 * sp_secs / few, "value": wl.R * few / sp_secs,
                              "unit": "verified tokens/s", "launches_per_call": int((ctx.launch_count() - l1) // few),
                              "bound": "tensor", "achieved": fl * few / sp_secs / 1e12, "peak": peaks["tflops_sustained"],
                              "roofline_unit": "TFLOP/s", "frac": fl * few / sp_secs / 1e12 / peaks["tflops_sustained"]}

    # Bonus token of the all-accepted branch of Alg. 1 folded into the round (the target chain runs R + B rows), against
    # the plain round on the same inputs; and a round under the DDIM-100 sampler of the paper's sampler table (100 of
    # 1000 linear-beta steps, eta = 1: same kernels, other coefficients and feature rows).
    if full and world == 1 and not args.no_seq:
        r0 = rounds[0]
        nxt = gen.make_round_inputs(gen.Workload(**{**wl.__dict__, "gamma": 1}), seed_offset=321, weights=False)
        zn, xn, en = (torch.from_numpy(a).to(dev) for a in (nxt.z_p, nxt.x_T, nxt.eps))
        xb = torch.zeros(wl.B, r0.C, dtype=torch.float32, device=dev)
        tk = torch.zeros(wl.B, dtype=torch.int32, device=dev)
        bonus_step = lambda i: ctx.csd_round_bonus(r0.head_q, r0.head_p, r0.sched_q, r0.sched_p, wl.B, wl.gamma, wl.cfg,
                                                   wl.cfg_scale, wl.cap, r0.z_q, r0.z_p, r0.x_T, r0.eps, r0.u, r0.xi, r0.v,
                                                   zn, xn, en, r0.x0, r0.mu1_q, r0.mu1_p, r0.logratio, r0.n_accept,
                                                   r0.accept_mask, r0.x_new, r0.n_prop, r0.flags, r0.cap_hits, xb, tk)
        plain_step = lambda i: r0.fused_round()
        timed(bonus_step, 3); b_secs = timed(bonus_step, few)
        timed(plain_step, 3); p_secs = timed(plain_step, few)
        out["bonus_fused_tail"] = {"call": "csd_round_bonus", "ms_per_round": 1e3 * b_secs / few,
                                   "plain_round_ms": 1e3 * p_secs / few, "extra_frac": b_secs / p_secs - 1.0,
                                   "extra_rows": f"{wl.B} of {wl.R} token rows"}
        if wl.T == 100:
            N = 1000
            steps_d = np.linspace(N // wl.T, N, wl.T).astype(np.int64)
            inp_d = gen.make_round_inputs(wl, seed_offset=777, weights=False)
            inp_d.w_q, inp_d.w_p = inp0.w_q, inp0.w_p
            inp_d.tfeat = np.ascontiguousarray(gen.timestep_features(N, wl.draft.F)[steps_d - 1])
            co = api.ddim_coefficients(gen.beta_linear(N), steps_d, 1.0)
            rd = DeviceRound(inp_d, ctx=ctx, device=local, heads=(r0.head_q, r0.head_p), coeffs_q=co, coeffs_p=co)
            ddim_step = lambda i: rd.fused_round()
            timed(ddim_step, 3); d_secs = timed(ddim_step, few)
            out["ddim100"] = {"sampler": "DDIM, 100 of 1000 linear-beta steps, eta = 1", "ms_per_round": 1e3 * d_secs / few,
                              "value": wl.R * few / d_secs, "unit": UNIT}

    # per-kernel-class device time (events around every launch: separate pass).  The three calls one after the
    # other: the same kernels and grids as csd_round, but the draft and the target chain do not share the GPU,
    # so a launch's duration is the kernel's own
    if full and not args.no_profile:
        ctx.profile(True)
        timed(lambda i: rounds[i % nsets].three_calls(), 3)
        out["prof"] = ctx.profile_read()
        ctx.profile(False)
    ctx.close()
    del flush
    torch.cuda.empty_cache()
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2411_11925_b200 import inputs as gen

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    wl = gen.WORKLOADS[args.workload]
    peaks = load_peaks()
    rps = args.rounds_per_step if args.rounds_per_step > 0 else max(1, wl.tokens // wl.gamma)
    m = measure(args.workload, args, peaks, args.steps, args.warmup, rps, full=True)
    secs, e2e_secs = m["secs"], m["e2e_secs"]
    if world > 1:
        t = torch.tensor([secs, e2e_secs], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        secs, e2e_secs = float(t[0]), float(t[1])
    tokens = wl.R * m["rounds"] * world
    value = tokens / secs

    # short runs of the other workloads (single rounds, an L2 flush between them): one line carries them all
    others = {}
    if world == 1 and not args.no_workloads:
        for name in gen.WORKLOADS:
            if name == args.workload:
                continue
            o = measure(name, args, peaks, 5, 3, 1, full=False)
            w = o["wl"]
            tf = w.flops_per_round() * o["rounds"] / o["secs"] / 1e12
            ent = {"ms_per_round": 1e3 * o["secs"] / o["rounds"], "value": w.R * o["rounds"] / o["secs"], "unit": UNIT,
                   "rounds_timed": o["rounds"], "B": w.B, "gamma": w.gamma, "T": w.T,
                   "draft_head": f"{w.draft.L}x{w.draft.W}", "target_head": f"{w.target.L}x{w.target.W}",
                   "operands": w.operand_format, "algorithmic_tflops": tf,
                   "sm_mhz": o["clocks"]["sm_mhz"], "clock_reasons": o["clocks"]["reasons"], "decisions": o["decisions"]}
            if w.operand_format != "f32":
                ent["path_frac_of_tensor_peak"] = tf / peaks["tflops_sustained"]
            if "single_path" in o:
                ent["single_path"] = {k: o["single_path"][k] for k in ("ms", "achieved", "frac")}
            if "prefill" in o:
                ent["prefill"] = o["prefill"]
            others[name] = ent

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None,
                "dtype": {"f16": "f16 (bf16-valued weights, fp32 accumulate)", "bf16": "bf16", "f32": "f32"}[wl.operand_format],
                "data": "synthetic",
                "config": {"workload": wl.name, "B_per_gpu": wl.B, "gamma": wl.gamma, "T": wl.T, "cfg_scale": wl.cfg_scale,
                           "draft_head": f"{wl.draft.L}x{wl.draft.W} (z {wl.draft.Dz})",
                           "target_head": f"{wl.target.L}x{wl.target.W} (z {wl.target.Dz})",
                           "rounds_per_step": rps,
                           "step": f"{rps} speculative rounds = {rps * wl.gamma} tokens per sequence "
                                   f"(one image-shaped pass), fresh z / noise / uniforms from 3 rotating input sets",
                           "parallelism": f"sequences sharded over {world} GPU(s), heads replicated, no collective",
                           "l2": "256 MB L2 flush between timed steps (outside the per-step event pairs)",
                           "call": "csd_round"},
                "ms_per_round": 1e3 * secs / m["rounds"],
                "clocks": m["clocks"],
                "e2e": {"value": tokens / e2e_secs, "unit": UNIT, "h2d_bytes_per_step": int(m.get("h2d", 0)),
                        "d2h_bytes_per_step": int(m.get("d2h", 0)), "call": "csd_round_host (pinned host buffers)"},
                "gpu_launches": int(m["launches"])}
        tf = wl.flops_per_round() * m["rounds"] / secs / 1e12
        line["algorithmic_tflops"] = tf
        line["path_frac_of_tensor_peak"] = tf / peaks["tflops_sustained"]
        line["decisions"] = m["decisions"]
        prof = m.get("prof")
        ch = m.get("chains")
        if ch and ch["persistent_chain_kernel"] and wl.operand_format != "f32":
            # the dominant kernel of the timed region is the target chain's persistent kernel: one launch per csd_verify
            # call, timed by events around the call on the library's stream (the other kernels of the call take microseconds)
            nb0 = -(-wl.R // (64 if wl.cfg else 128))
            ctas = 8 * (nb0 + (nb0 & 1))            # one CTA per 128 x 128 tile of a layer, row blocks paired
            fl = wl.Rh * wl.T * wl.target.flops_per_row_step()
            ach = fl / (ch["verify_ms"] * 1e-3) / 1e12
            line["roofline"] = {"bound": "tensor", "kernel": "pchain_kernel (target chain, one launch per call)",
                                "achieved": ach, "peak": peaks["tflops_sustained"], "unit": "TFLOP/s",
                                "frac": ach / peaks["tflops_sustained"],
                                "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get((wl.name, "pchain_target")),
                                "peak_source": f"{peaks['source']} bf16 sustained (fp16 has the same nominal rate)",
                                "avg_launch_us": 1e3 * ch["verify_ms"], "flops_per_launch": fl,
                                "sms_used": f"{ctas} of 148 (the draft chain's kernel runs beside it on others)",
                                "draft_chain": {"avg_launch_us": 1e3 * ch["draft_ms"],
                                                "achieved": wl.Rh * wl.T * wl.draft.flops_per_row_step() / (ch["draft_ms"] * 1e-3) / 1e12}}
            line["chains"] = ch
        elif prof:
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
        if prof and "roofline" in line and "per_class" not in line["roofline"]:
            tot_ms = sum(v["ms"] for v in prof.values())
            line["layer_kernels_per_class"] = {k: {"launches": v["launches"], "ms": round(v["ms"], 3), "share": round(v["ms"] / tot_ms, 4),
                                                    "tflops": (v["flops"] / (v["ms"] * 1e-3) / 1e12 if v["ms"] > 0 else 0.0)}
                                               for k, v in prof.items()}
        for k in ("sequential_draft", "prefill", "single_path", "bonus_fused_tail", "ddim100"):
            if k in m:
                line[k] = m[k]
        if others:
            line["workloads"] = others
        if not args.no_cpu_baseline and world == 1:
            val, threads, desc, times, ref = time_oracle(args.workload)
            line["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc,
                                    "runs": len(times)}
            nseq = min(wl.B, SAMPLE_SEQS.get(args.workload, 1))
            line["checker_comparison"] = checker_counts(m["res0"], ref, m["inp0"].u, wl, nseq)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    a = parse_args()
    cmd = reexec_argv(a, sys.argv[1:])
    if cmd is not None:
        os.execv(cmd[0], cmd)
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
