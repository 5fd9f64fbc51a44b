"""Convenience driver over the C-ABI binding: uploads one round of inputs, owns
the output tensors and calls the library (marshalling only, no arithmetic)."""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

from . import api
from .inputs import RoundInputs


class DeviceRound:
    """Device-resident heads, schedules, inputs and outputs of one speculative round."""

    def __init__(self, inp: RoundInputs, ctx: Optional[api.Context] = None, device: int = 0,
                 heads: Optional[tuple] = None, tau_q: Optional[float] = None, tau_p: Optional[float] = None,
                 coeffs_q: Optional[dict] = None, coeffs_p: Optional[dict] = None):
        """coeffs_q / coeffs_p: transition coefficients {"a", "b", "sigma"} to use instead of the DDPM ones of
        inp.beta (for instance api.ddim_coefficients); inp.tfeat must then hold the rows of the same timesteps."""
        wl = inp.wl
        self.inp, self.wl = inp, wl
        self.dev = torch.device("cuda", device)
        self.ctx = ctx or api.Context(device)
        if heads is None:
            self.head_q = api.Head(self.ctx, inp.w_q, wl.operand_format)
            self.head_p = api.Head(self.ctx, inp.w_p, wl.operand_format)
        else:
            self.head_q, self.head_p = heads
        self.tfeat = torch.from_numpy(inp.tfeat).to(self.dev)
        cq = coeffs_q or api.ddpm_coefficients(inp.beta, wl.tau if tau_q is None else tau_q)
        cp = coeffs_p or api.ddpm_coefficients(inp.beta, wl.tau if tau_p is None else tau_p)
        self.sched_q = api.Schedule(cq["a"], cq["b"], cq["sigma"], self.tfeat)
        self.sched_p = api.Schedule(cp["a"], cp["b"], cp["sigma"], self.tfeat)
        self.C = wl.draft.C
        self.upload(inp)
        B, R, Cd = wl.B, wl.R, self.C
        f32 = dict(dtype=torch.float32, device=self.dev)
        self.x0, self.mu1_q, self.mu1_p, self.x1_q = (torch.zeros(R, Cd, **f32) for _ in range(4))
        self.logratio = torch.zeros(B, wl.gamma, **f32)
        self.n_accept = torch.zeros(B, dtype=torch.int32, device=self.dev)
        self.accept_mask = torch.zeros(B, dtype=torch.int32, device=self.dev)
        self.x_new = torch.zeros(B, Cd, **f32)
        self.n_prop = torch.zeros(B, dtype=torch.int32, device=self.dev)
        self.flags = torch.zeros(B, dtype=torch.int32, device=self.dev)
        self.cap_hits = torch.zeros(1, dtype=torch.int32, device=self.dev)

    def upload(self, inp: RoundInputs):
        to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(self.dev)
        self.z_q, self.z_p, self.x_T, self.eps = to(inp.z_q), to(inp.z_p), to(inp.x_T), to(inp.eps)
        self.u, self.xi, self.v = to(inp.u), to(inp.xi), to(inp.v)

    @property
    def log_sigma(self) -> float:
        return self.sched_q.log_sigma_term(self.sched_p, self.C)

    def draft(self):
        wl = self.wl
        self.ctx.csd_draft_denoise(self.head_q, self.sched_q, wl.R, wl.cfg, wl.cfg_scale, self.z_q, self.x_T,
                                   self.eps, self.x0, self.mu1_q, self.x1_q)

    def verify(self):
        wl = self.wl
        self.ctx.csd_verify(self.head_p, self.sched_p, self.sched_q, wl.B, wl.gamma, wl.cfg, wl.cfg_scale,
                            self.z_p, self.x_T, self.eps, self.x0, self.mu1_q, self.u, self.logratio,
                            self.n_accept, self.accept_mask, self.mu1_p)

    def resample(self):
        wl = self.wl
        self.ctx.csd_resample(wl.B, wl.gamma, self.C, wl.cap, self.log_sigma, float(self.sched_p.sigma[0]),
                              float(self.sched_q.sigma[0]), self.n_accept, self.mu1_p, self.mu1_q, self.xi,
                              self.v, self.x_new, self.n_prop, self.flags, self.cap_hits)

    def draft_traj(self):
        """Draft trajectories with every state and mean recorded (input of the single-path ratio, Eq. 2)."""
        wl = self.wl
        if not hasattr(self, "traj_x"):
            T = len(self.sched_q.sigma)
            self.traj_x = torch.zeros(T + 1, wl.R, self.C, dtype=torch.float32, device=self.dev)
            self.traj_mu = torch.zeros(T, wl.R, self.C, dtype=torch.float32, device=self.dev)
        self.ctx.csd_draft_denoise_traj(self.head_q, self.sched_q, wl.R, wl.cfg, wl.cfg_scale, self.z_q, self.x_T,
                                        self.eps, self.traj_x, self.traj_mu)

    def verify_single_path(self, steps_per_pass: int = 0, traj_x=None, traj_mu=None, mu_p_traj=None):
        wl = self.wl
        self.ctx.csd_verify_single_path(self.head_p, self.sched_p, self.sched_q, wl.B, wl.gamma, wl.cfg, wl.cfg_scale,
                                        self.z_p, self.traj_x if traj_x is None else traj_x,
                                        self.traj_mu if traj_mu is None else traj_mu, self.u, steps_per_pass,
                                        self.logratio, self.n_accept, self.accept_mask, mu_p_traj)

    def verify_unaligned(self, eps_p):
        """csd_verify with the target's own noise eps_p (no trajectory alignment)."""
        wl = self.wl
        self.ctx.csd_verify_unaligned(self.head_p, self.sched_p, self.sched_q, wl.B, wl.gamma, wl.cfg, wl.cfg_scale,
                                      self.z_p, self.x_T, eps_p, self.eps, self.x0, self.mu1_q, self.u, self.logratio,
                                      self.n_accept, self.accept_mask, self.mu1_p)

    def three_calls(self):
        self.draft(); self.verify(); self.resample()

    def _round_args(self, host: Optional[dict] = None):
        wl = self.wl
        t = host or self.__dict__
        return (self.head_q, self.head_p, self.sched_q, self.sched_p, wl.B, wl.gamma, wl.cfg, wl.cfg_scale, wl.cap,
                t["z_q"], t["z_p"], t["x_T"], t["eps"], t["u"], t["xi"], t["v"], t["x0"], t["mu1_q"], t["mu1_p"],
                t["logratio"], t["n_accept"], t["accept_mask"], t["x_new"], t["n_prop"], t["flags"], t["cap_hits"])

    def fused_round(self):
        self.ctx.csd_round(*self._round_args())

    def make_host_buffers(self) -> dict:
        """Pinned host copies of every input and output, for csd_round_host."""
        names = ("z_q", "z_p", "x_T", "eps", "u", "xi", "v", "x0", "mu1_q", "mu1_p", "logratio", "n_accept",
                 "accept_mask", "x_new", "n_prop", "flags", "cap_hits")
        return {n: getattr(self, n).cpu().pin_memory() for n in names}

    def host_round(self, host: dict):
        self.ctx.csd_round_host(*self._round_args(host))

    def results(self, host: Optional[dict] = None) -> Dict[str, np.ndarray]:
        self.ctx.sync()
        t = host or self.__dict__
        get = lambda n: (t[n].cpu().numpy().copy() if isinstance(t[n], torch.Tensor) else np.array(t[n]))
        out = {n: get(n) for n in ("x0", "mu1_q", "mu1_p", "logratio", "n_accept", "accept_mask", "x_new", "n_prop",
                                   "flags", "cap_hits")}
        if host is None:
            out["x1_q"] = get("x1_q")
        return out
