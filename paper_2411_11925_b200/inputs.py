"""Seeded synthetic inputs for continuous speculative decoding workloads.

This module only *draws and shapes data*: head weights, condition vectors z,
reparameterization noise, uniforms, the beta ladder and the timestep feature
table.  It contains none of the method's arithmetic (no head forward, no DDPM
coefficients, no densities), so both the CUDA library's tests and the CPU
checker can consume the very same arrays without sharing any computation.

Workloads are stand-ins, by shape only, for the MAR / Harmon style 256x256
(256 latent tokens of dim 16) and 512x512 (1024 tokens of dim 16) settings of
the paper's experiments (Sec. 4 "Implementation Details"); no dataset or
trained checkpoint is involved.

Head parameter naming (one head, width W, L residual blocks, condition dim Dz,
token dim C, timestep feature dim F); every matrix is row-major [out, in]:

    Wz[W,Dz] bz[W]           condition projection
    Wt1[W,F] bt1[W]          timestep MLP, first layer
    Wt2[W,W] bt2[W]          timestep MLP, second layer
    Win[W,C] bin[W]          input projection
    Wada[L,3W,W] bada[L,3W]  per-block AdaLN (shift | scale | gate)
    W1[L,W,W] b1[L,W]        per-block MLP, first layer
    W2[L,W,W] b2[L,W]        per-block MLP, second layer
    Wfada[2W,W] bfada[2W]    final AdaLN (shift | scale)
    Wout[C,W] bout[C]        output projection ([2C,W], [2C] for a head that also predicts its
                             transition's variance: rows C..2C give the variance parameter)
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

SEED_BASE = 2411119250

WEIGHT_NAMES = (
    "Wz", "bz", "Wt1", "bt1", "Wt2", "bt2", "Win", "bin",
    "Wada", "bada", "W1", "b1", "W2", "b2", "Wfada", "bfada", "Wout", "bout",
)


@dataclass(frozen=True)
class HeadSpec:
    """Shape of one diffusion head."""
    L: int
    W: int
    Dz: int
    C: int = 16
    F: int = 256
    var_out: bool = False   # the head has 2C outputs: eps_hat and a variance parameter per coordinate

    def n_params(self) -> int:
        W, L, Dz, C, F = self.W, self.L, self.Dz, self.C, self.F
        Co = 2 * C if self.var_out else C
        return (W * Dz + W + W * F + W + W * W + W + W * C + W
                + L * (3 * W * W + 3 * W) + 2 * L * (W * W + W)
                + 2 * W * W + 2 * W + Co * W + Co)

    def flops_per_row_step(self) -> float:
        """Algorithmic FLOPs of one head evaluation for one head row:
        2*(C*W + L*5*W^2 + 2*W^2 + W*C)."""
        W, L, C = self.W, self.L, self.C
        return 2.0 * (C * W + L * 5 * W * W + 2 * W * W + W * C)


@dataclass(frozen=True)
class Workload:
    """One synthetic workload (a row of the configuration table)."""
    name: str
    index: int
    B: int
    gamma: int
    T: int
    cfg: bool
    cfg_scale: float
    draft: HeadSpec
    target: HeadSpec
    bf16: bool
    tau: float = 1.0
    cap: int = 64
    tokens: int = 256
    prefill: int = 0
    perturb_std: float = 0.0   # >0: draft = target weights + N(0, std^2)
    operand: str = ""          # GEMM operand format: "f32" | "bf16" | "f16"; "" = "f16" if bf16 else "f32"

    @property
    def operand_format(self) -> str:
        """bf16=True means the weight and z VALUES are bf16-representable; by default such a
        workload runs with fp16 tensor-core operands (those values are exact in fp16)."""
        return self.operand or ("f16" if self.bf16 else "f32")

    @property
    def R(self) -> int:
        return self.B * self.gamma

    @property
    def Rh(self) -> int:
        return self.R * (2 if self.cfg else 1)

    def flops_per_round(self) -> float:
        return self.Rh * self.T * (self.draft.flops_per_row_step()
                                   + self.target.flops_per_row_step())


WORKLOADS: Dict[str, Workload] = {
    "tiny_fp32": Workload("tiny_fp32", 0, B=1, gamma=4, T=10, cfg=False, cfg_scale=1.0,
                          draft=HeadSpec(1, 128, 256), target=HeadSpec(2, 256, 256),
                          bf16=False, tokens=4),
    "mar256": Workload("mar256", 1, B=64, gamma=8, T=100, cfg=True, cfg_scale=3.0,
                       draft=HeadSpec(3, 1024, 768), target=HeadSpec(6, 1024, 1024),
                       bf16=True, tokens=256),
    "large_target": Workload("large_target", 2, B=128, gamma=16, T=100, cfg=True, cfg_scale=3.0,
                             draft=HeadSpec(6, 1024, 1024), target=HeadSpec(12, 1536, 1280),
                             bf16=True, tokens=256, prefill=16),
    "mar512": Workload("mar512", 3, B=32, gamma=32, T=100, cfg=True, cfg_scale=3.0,
                       draft=HeadSpec(6, 1024, 1024), target=HeadSpec(12, 1536, 1280),
                       bf16=True, tokens=1024),
    "ar_stress": Workload("ar_stress", 4, B=256, gamma=16, T=50, cfg=False, cfg_scale=1.0,
                          draft=HeadSpec(8, 1024, 1024), target=HeadSpec(8, 1024, 1024),
                          bf16=True, tokens=256, perturb_std=0.05),
}


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even) and return
    them as float32, so that a later cast to bf16 anywhere is exact."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) & np.uint32(0xFFFF0000)).view(np.float32)


def beta_linear(T: int, lo: float = 1e-4, hi: float = 0.02) -> np.ndarray:
    """The linear beta ladder of a T-step DDPM, beta_1..beta_T (float64)."""
    return np.linspace(lo, hi, T, dtype=np.float64)


def timestep_features(T: int, F: int = 256, max_period: float = 10000.0) -> np.ndarray:
    """Sinusoidal feature table [T, F] (float32); row t-1 belongs to timestep t.
    It is an *input* of the head: both implementations read this table."""
    half = F // 2
    freqs = np.exp(-np.log(max_period) * np.arange(half, dtype=np.float64) / half)
    t = np.arange(1, T + 1, dtype=np.float64)[:, None]
    ang = t * freqs[None, :]
    return np.concatenate([np.cos(ang), np.sin(ang)], axis=1).astype(np.float32)


def _xavier(rng: np.random.Generator, *shape: int) -> np.ndarray:
    fan_out, fan_in = shape[-2], shape[-1]
    bound = np.sqrt(6.0 / (fan_in + fan_out))
    return rng.uniform(-bound, bound, size=shape).astype(np.float32)


def _normal(rng: np.random.Generator, std: float, *shape: int) -> np.ndarray:
    return (std * rng.standard_normal(size=shape)).astype(np.float32)


def make_head_weights(spec: HeadSpec, rng: np.random.Generator, bf16: bool = False
                      ) -> Dict[str, np.ndarray]:
    """Random-init head: Xavier-uniform for the block / AdaLN / in / out
    matrices, N(0, 0.02^2) for Wz, Wt1, Wt2 and every bias.  No layer is
    zero-initialised (a zero gate would make every test vacuous)."""
    W, L, Dz, C, F = spec.W, spec.L, spec.Dz, spec.C, spec.F
    Co = 2 * C if spec.var_out else C
    w = {
        "Wz": _normal(rng, 0.02, W, Dz), "bz": _normal(rng, 0.02, W),
        "Wt1": _normal(rng, 0.02, W, F), "bt1": _normal(rng, 0.02, W),
        "Wt2": _normal(rng, 0.02, W, W), "bt2": _normal(rng, 0.02, W),
        "Win": _xavier(rng, W, C), "bin": _normal(rng, 0.02, W),
        "Wada": _xavier(rng, L, 3 * W, W), "bada": _normal(rng, 0.02, L, 3 * W),
        "W1": _xavier(rng, L, W, W), "b1": _normal(rng, 0.02, L, W),
        "W2": _xavier(rng, L, W, W), "b2": _normal(rng, 0.02, L, W),
        "Wfada": _xavier(rng, 2 * W, W), "bfada": _normal(rng, 0.02, 2 * W),
        "Wout": _xavier(rng, Co, W), "bout": _normal(rng, 0.02, Co),
    }
    if bf16:
        w = {k: (round_to_bf16(v) if v.ndim >= 2 and k.startswith("W") else v) for k, v in w.items()}
    return w


def perturb_head_weights(w: Dict[str, np.ndarray], rng: np.random.Generator, std: float,
                         bf16: bool = False) -> Dict[str, np.ndarray]:
    """A second head = the given one plus N(0, std^2) noise on every parameter."""
    out = {}
    for k in WEIGHT_NAMES:
        v = w[k] + (std * rng.standard_normal(size=w[k].shape)).astype(np.float32)
        if bf16 and k.startswith("W"):
            v = round_to_bf16(v)
        out[k] = v.astype(np.float32)
    return out


@dataclass
class RoundInputs:
    """Everything one speculative round consumes."""
    wl: Workload
    w_q: Dict[str, np.ndarray]
    w_p: Dict[str, np.ndarray]
    z_q: np.ndarray        # [Rh, Dz_q]  rows [cond | uncond]
    z_p: np.ndarray        # [Rh, Dz_p]
    x_T: np.ndarray        # [R, C]
    eps: np.ndarray        # [T, R, C]   slice t-1 is the noise of step t
    u: np.ndarray          # [B, gamma]  accept uniforms in (0,1)
    xi: np.ndarray         # [B, cap, C] resample proposals' normals
    v: np.ndarray          # [B, cap]    resample uniforms in (0,1)
    beta: np.ndarray       # [T] float64
    tfeat: np.ndarray      # [T, F] float32
    extras: dict = field(default_factory=dict)


def _open_uniform(rng: np.random.Generator, *shape: int) -> np.ndarray:
    x = rng.random(size=shape).astype(np.float32)
    tiny = np.float32(2.0 ** -24)
    return np.clip(x, tiny, np.float32(1.0) - tiny)


def make_round_inputs(wl: Workload, B: Optional[int] = None, seed_offset: int = 0,
                      weights: bool = True) -> RoundInputs:
    """Draw one round of inputs for `wl` from PCG64(SEED_BASE + index + seed_offset)
    in the fixed order weights_q, weights_p, z_q, z_p, x_T, eps, u, xi, v.
    `B` overrides the batch (used by parity tests that run fewer sequences)."""
    if B is not None and B != wl.B:
        wl = Workload(**{**wl.__dict__, "B": B})
    rng = np.random.Generator(np.random.PCG64(SEED_BASE + wl.index + seed_offset))
    if weights:
        if wl.perturb_std > 0.0:
            w_p = make_head_weights(wl.target, rng, wl.bf16)
            w_q = perturb_head_weights(w_p, rng, wl.perturb_std, wl.bf16)
        else:
            w_q = make_head_weights(wl.draft, rng, wl.bf16)
            w_p = make_head_weights(wl.target, rng, wl.bf16)
    else:
        w_q, w_p = {}, {}
    R, Rh, C, T = wl.R, wl.Rh, wl.draft.C, wl.T
    z_q = rng.standard_normal(size=(Rh, wl.draft.Dz)).astype(np.float32)
    z_p = rng.standard_normal(size=(Rh, wl.target.Dz)).astype(np.float32)
    if wl.bf16:
        z_q, z_p = round_to_bf16(z_q), round_to_bf16(z_p)
    x_T = rng.standard_normal(size=(R, C)).astype(np.float32)
    eps = rng.standard_normal(size=(T, R, C)).astype(np.float32)
    u = _open_uniform(rng, wl.B, wl.gamma)
    xi = rng.standard_normal(size=(wl.B, wl.cap, C)).astype(np.float32)
    v = _open_uniform(rng, wl.B, wl.cap)
    return RoundInputs(wl, w_q, w_p, z_q, z_p, x_T, eps, u, xi, v,
                       beta_linear(T), timestep_features(T, wl.draft.F))


def select_sequences(inp: RoundInputs, seqs) -> RoundInputs:
    """Restrict a round to the given sequence indices (rows are independent, so a
    checker may evaluate only some sequences of a large batch)."""
    wl = inp.wl
    seqs = np.asarray(list(seqs), dtype=np.int64)
    g, R = wl.gamma, wl.R
    rows = (seqs[:, None] * g + np.arange(g)[None, :]).reshape(-1)
    hrows = np.concatenate([rows, rows + R]) if wl.cfg else rows
    sub = Workload(**{**wl.__dict__, "B": len(seqs)})
    return RoundInputs(sub, inp.w_q, inp.w_p, inp.z_q[hrows], inp.z_p[hrows], inp.x_T[rows],
                       inp.eps[:, rows], inp.u[seqs], inp.xi[seqs], inp.v[seqs],
                       inp.beta, inp.tfeat, {"rows": rows, "seqs": seqs})


def shard_sequences(B: int, world: int, rank: int) -> range:
    """Contiguous block of sequence indices owned by `rank` when B sequences are split over
    `world` ranks (the first B % world ranks get one more).  Rows of different sequences never
    interact, so a sharded round needs no exchange."""
    base, extra = divmod(B, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))
