"""ctypes binding of libcsd.so: argument marshalling only.

Every step of the hot path runs inside the CUDA library; this module passes
pointers and sizes.  torch is used for device memory and streams.  There is no
CPU path: importing this module raises if the library is missing.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np
import torch

from . import build as _build

_c_float_p = C.POINTER(C.c_float)

ERRORS = {0: "CSD_OK", -1: "CSD_ERR_INVALID_ARG", -2: "CSD_ERR_SHAPE", -3: "CSD_ERR_UNSUPPORTED",
          -4: "CSD_ERR_WORKSPACE", -5: "CSD_ERR_CUDA", -6: "CSD_ERR_TIMEOUT", -7: "CSD_ERR_NONFINITE"}
CSD_F32, CSD_BF16, CSD_F16 = 0, 1, 2
DTYPES = {"f32": CSD_F32, "bf16": CSD_BF16, "f16": CSD_F16}

EXPORTS = ("csd_create", "csd_destroy", "csd_last_error", "csd_sync", "csd_launch_count",
           "csd_set_chain_mode", "csd_profile", "csd_profile_read", "csd_set_wait_limit", "csd_selftest_wait_timeout",
           "csd_schedule_ddpm", "csd_schedule_ddim", "csd_log_sigma_term", "csd_schedule_lv_ddpm",
           "csd_draft_denoise_lv", "csd_verify_lv", "csd_resample_lv", "csd_round_lv",
           "csd_head_create", "csd_head_destroy", "csd_draft_denoise", "csd_draft_denoise_static", "csd_verify",
           "csd_accept_scan", "csd_resample", "csd_round", "csd_round_host", "csd_draft_denoise_traj",
           "csd_verify_single_path", "csd_verify_unaligned", "csd_bonus_token", "csd_verify_bonus", "csd_round_bonus",
           "csd_gmm_draft_sample", "csd_gmm_verify", "csd_gmm_resample")

WEIGHT_FIELDS = ("Wz", "bz", "Wt1", "bt1", "Wt2", "bt2", "Win", "bin", "Wada", "bada",
                 "W1", "b1", "W2", "b2", "Wfada", "bfada", "Wout", "bout")


class CsdError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"{ERRORS.get(code, code)}: {msg}")
        self.code = code


class _HeadDesc(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("C", "W", "L", "Dz", "F", "dtype", "var_out")]


class _HeadWeights(C.Structure):
    _fields_ = [(n, _c_float_p) for n in WEIGHT_FIELDS]


class _Schedule(C.Structure):
    _fields_ = [("T", C.c_int), ("a", _c_float_p), ("b", _c_float_p), ("sigma", _c_float_p),
                ("tfeat", C.c_void_p)]


class _Gmm(C.Structure):
    _fields_ = [("K", C.c_int), ("logw", C.c_void_p), ("mu", C.c_void_p), ("log_sigma", C.c_void_p)]


class _ScheduleLV(C.Structure):
    _fields_ = [("T", C.c_int), ("a", _c_float_p), ("b", _c_float_p), ("lv_min", _c_float_p), ("lv_max", _c_float_p),
                ("tfeat", C.c_void_p)]


def load_library(path: Optional[str] = None) -> C.CDLL:
    path = path or _build.LIB_PATH
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run `python -m paper_2411_11925_b200.build` "
                          "(or __graft_entry__.build()); there is no CPU fallback")
    lib = C.CDLL(path)
    vp, i32, f32, f64 = C.c_void_p, C.c_int, C.c_float, C.c_double
    lib.csd_create.argtypes = [C.POINTER(vp), i32, vp]
    lib.csd_destroy.argtypes = [vp]
    lib.csd_last_error.argtypes = [vp]; lib.csd_last_error.restype = C.c_char_p
    lib.csd_sync.argtypes = [vp]
    lib.csd_launch_count.argtypes = [vp]; lib.csd_launch_count.restype = C.c_int64
    lib.csd_set_chain_mode.argtypes = [vp, C.c_int]
    lib.csd_set_wait_limit.argtypes = [vp, C.c_int64]
    lib.csd_selftest_wait_timeout.argtypes = [vp]
    f64p, i32p = C.POINTER(f64), C.POINTER(C.c_int32)
    lib.csd_schedule_ddpm.argtypes = [i32, f64p, f64, _c_float_p, _c_float_p, _c_float_p]
    lib.csd_schedule_ddim.argtypes = [i32, f64p, i32, i32p, f64, _c_float_p, _c_float_p, _c_float_p]
    lib.csd_log_sigma_term.argtypes = [i32, _c_float_p, _c_float_p, i32, f64p]
    lib.csd_schedule_lv_ddpm.argtypes = [i32, f64p, f64] + [_c_float_p] * 4
    lib.csd_draft_denoise_lv.argtypes = [vp, vp, C.POINTER(_ScheduleLV), i32, i32, f32] + [vp] * 8
    lib.csd_verify_lv.argtypes = [vp, vp, C.POINTER(_ScheduleLV), i32, i32, i32, f32] + [vp] * 15
    lib.csd_resample_lv.argtypes = [vp, i32, i32, i32, i32] + [vp] * 12
    lib.csd_round_lv.argtypes = ([vp, vp, vp, C.POINTER(_ScheduleLV), C.POINTER(_ScheduleLV), i32, i32, i32, f32, i32]
                                 + [vp] * 22)
    gp = C.POINTER(_Gmm)
    lib.csd_gmm_draft_sample.argtypes = [vp, i32, i32, gp] + [vp] * 4
    lib.csd_gmm_verify.argtypes = [vp, i32, i32, i32, gp, gp] + [vp] * 5
    lib.csd_gmm_resample.argtypes = [vp, i32, i32, i32, i32, gp, gp] + [vp] * 8
    lib.csd_profile.argtypes = [vp, i32]
    lib.csd_profile_read.argtypes = [vp, i32, C.POINTER(C.c_int64), C.POINTER(f64), C.POINTER(f64)]
    lib.csd_head_create.argtypes = [vp, C.POINTER(_HeadDesc), C.POINTER(_HeadWeights), C.POINTER(vp)]
    lib.csd_head_destroy.argtypes = [vp]
    lib.csd_draft_denoise.argtypes = [vp, vp, C.POINTER(_Schedule), i32, i32, f32] + [vp] * 6
    lib.csd_draft_denoise_static.argtypes = lib.csd_draft_denoise.argtypes
    lib.csd_verify.argtypes = [vp, vp, C.POINTER(_Schedule), C.POINTER(_Schedule), i32, i32, i32, f32] + [vp] * 10
    lib.csd_draft_denoise_traj.argtypes = [vp, vp, C.POINTER(_Schedule), i32, i32, f32] + [vp] * 5
    lib.csd_verify_single_path.argtypes = ([vp, vp, C.POINTER(_Schedule), C.POINTER(_Schedule), i32, i32, i32, f32]
                                           + [vp] * 4 + [i32] + [vp] * 4)
    lib.csd_verify_unaligned.argtypes = ([vp, vp, C.POINTER(_Schedule), C.POINTER(_Schedule), i32, i32, i32, f32]
                                         + [vp] * 11)
    lib.csd_bonus_token.argtypes = [vp, vp, C.POINTER(_Schedule), i32, i32, i32, f32] + [vp] * 6
    lib.csd_verify_bonus.argtypes = [vp, vp, C.POINTER(_Schedule), C.POINTER(_Schedule), i32, i32, i32, f32] + [vp] * 15
    lib.csd_round_bonus.argtypes = ([vp, vp, vp, C.POINTER(_Schedule), C.POINTER(_Schedule), i32, i32, i32, f32, i32]
                                    + [vp] * 22)
    lib.csd_accept_scan.argtypes = [vp, i32, i32, i32, f64, f32, f32] + [vp] * 7
    lib.csd_resample.argtypes = [vp, i32, i32, i32, i32, f64, f32, f32] + [vp] * 9
    round_args = [vp, vp, vp, C.POINTER(_Schedule), C.POINTER(_Schedule), i32, i32, i32, f32, i32] + [vp] * 17
    lib.csd_round.argtypes = round_args
    lib.csd_round_host.argtypes = round_args
    for name in EXPORTS:
        if name not in ("csd_last_error", "csd_launch_count"):
            getattr(lib, name).restype = C.c_int
    return lib


_LIB = load_library()


def _schedule_out(n: int):
    out = {k: np.zeros(n, dtype=np.float32) for k in ("a", "b", "sigma")}
    return out, [out[k].ctypes.data_as(_c_float_p) for k in ("a", "b", "sigma")]


def ddpm_coefficients(beta: np.ndarray, tau: float = 1.0) -> Dict[str, np.ndarray]:
    """csd_schedule_ddpm: coefficient arrays {"a", "b", "sigma"} of the T-step DDPM behind Eq. 3."""
    beta = np.ascontiguousarray(beta, dtype=np.float64)
    out, ptrs = _schedule_out(beta.size)
    rc = _LIB.csd_schedule_ddpm(int(beta.size), beta.ctypes.data_as(C.POINTER(C.c_double)), float(tau), *ptrs)
    if rc != 0:
        raise CsdError(rc, "csd_schedule_ddpm: beta must lie in (0, 1) and tau be positive")
    return out


def ddim_coefficients(beta_full: np.ndarray, steps, eta: float) -> Dict[str, np.ndarray]:
    """csd_schedule_ddim: coefficient arrays of a DDIM sampler with stochasticity eta in (0, 1] on the ascending
    sub-sequence `steps` (1-based timesteps) of a DDPM's ladder.  Entry k-1 is the k-th step counted from x_0; pass
    the feature-table rows of the same timesteps as tfeat."""
    beta_full = np.ascontiguousarray(beta_full, dtype=np.float64)
    steps = np.ascontiguousarray(list(steps), dtype=np.int32)
    out, ptrs = _schedule_out(steps.size)
    rc = _LIB.csd_schedule_ddim(int(beta_full.size), beta_full.ctypes.data_as(C.POINTER(C.c_double)), int(steps.size),
                                steps.ctypes.data_as(C.POINTER(C.c_int32)), float(eta), *ptrs)
    if rc != 0:
        raise ValueError("csd_schedule_ddim: eta must be in (0, 1] and steps ascending timesteps within 1..len(beta_full)")
    return out


def lv_ddpm_coefficients(beta: np.ndarray, tau: float = 1.0) -> Dict[str, np.ndarray]:
    """csd_schedule_lv_ddpm: {"a", "b", "lv_min", "lv_max"} of a DDPM whose head predicts its variances."""
    beta = np.ascontiguousarray(beta, dtype=np.float64)
    out = {k: np.zeros(beta.size, dtype=np.float32) for k in ("a", "b", "lv_min", "lv_max")}
    rc = _LIB.csd_schedule_lv_ddpm(int(beta.size), beta.ctypes.data_as(C.POINTER(C.c_double)), float(tau),
                                   *[out[k].ctypes.data_as(_c_float_p) for k in ("a", "b", "lv_min", "lv_max")])
    if rc != 0:
        raise CsdError(rc, "csd_schedule_lv_ddpm: beta must lie in (0, 1) and tau be positive")
    return out


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous(), "tensor must be contiguous"
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"], "array must be contiguous"
        return t.ctypes.data
    raise TypeError(type(t))


class Schedule:
    """Keeps the host coefficient arrays and the device feature table alive."""

    def __init__(self, a, b, sigma, tfeat: torch.Tensor):
        self.a = np.ascontiguousarray(a, dtype=np.float32)
        self.b = np.ascontiguousarray(b, dtype=np.float32)
        self.sigma = np.ascontiguousarray(sigma, dtype=np.float32)
        assert tfeat.is_cuda and tfeat.dtype == torch.float32 and tfeat.is_contiguous()
        self.tfeat = tfeat
        self.T = int(self.sigma.shape[0])
        self.c = _Schedule(self.T, self.a.ctypes.data_as(_c_float_p), self.b.ctypes.data_as(_c_float_p),
                           self.sigma.ctypes.data_as(_c_float_p), tfeat.data_ptr())

    def log_sigma_term(self, other_p: "Schedule", Cdim: int) -> float:
        """csd_log_sigma_term: log Sigma of Eq. 7 for (self = draft, other_p = target)."""
        out = C.c_double()
        rc = _LIB.csd_log_sigma_term(self.T, self.sigma.ctypes.data_as(_c_float_p),
                                     other_p.sigma.ctypes.data_as(_c_float_p), int(Cdim), C.byref(out))
        if rc != 0:
            raise CsdError(rc, "csd_log_sigma_term")
        return float(out.value)


class ScheduleLV:
    """csd_schedule_lv: keeps the host arrays and the device feature table alive."""

    def __init__(self, a, b, lv_min, lv_max, tfeat: torch.Tensor):
        self.a, self.b, self.lv_min, self.lv_max = (np.ascontiguousarray(x, dtype=np.float32) for x in (a, b, lv_min, lv_max))
        assert tfeat.is_cuda and tfeat.dtype == torch.float32 and tfeat.is_contiguous()
        self.tfeat = tfeat
        self.T = int(self.a.shape[0])
        self.c = _ScheduleLV(self.T, *[x.ctypes.data_as(_c_float_p) for x in (self.a, self.b, self.lv_min, self.lv_max)],
                             tfeat.data_ptr())


class Context:
    def __init__(self, device: int = 0, stream: Optional[torch.cuda.Stream] = None):
        self._h = C.c_void_p()
        self.device = device
        self.stream = stream
        sp = stream.cuda_stream if stream is not None else None
        rc = _LIB.csd_create(C.byref(self._h), device, sp)
        if rc != 0:
            raise CsdError(rc, "csd_create failed")
        self._heads = []

    def _check(self, rc: int):
        if rc != 0:
            raise CsdError(rc, _LIB.csd_last_error(self._h).decode())

    def sync(self):
        self._check(_LIB.csd_sync(self._h))

    def launch_count(self) -> int:
        return int(_LIB.csd_launch_count(self._h))

    CHAIN_LAYERS, CHAIN_SMALL_BATCH, CHAIN_LAYERS_PLAIN, CHAIN_LAYER_KERNELS = 0, 1, 2, 3

    def set_chain_mode(self, mode: int):
        """csd_set_chain_mode: CHAIN_LAYERS (default: the persistent chain kernel where it applies, else one kernel per
        layer with folded blocks where they apply), CHAIN_LAYER_KERNELS (never the persistent chain kernel),
        CHAIN_LAYERS_PLAIN (three kernels per block everywhere) or CHAIN_SMALL_BATCH (chains of at most 128 head rows
        run as one persistent kernel over the whole GPU)."""
        self._check(_LIB.csd_set_chain_mode(self._h, int(mode)))

    def set_wait_limit(self, cycles: int):
        self._check(_LIB.csd_set_wait_limit(self._h, int(cycles)))

    def selftest_wait_timeout(self):
        self._check(_LIB.csd_selftest_wait_timeout(self._h))

    KERNEL_CLASSES = ("cond_proj", "mlp1_silu", "adaln_modulate", "mlp2_gate_residual", "final_mod_outproj", "step", "chain")

    def profile(self, enable: bool):
        self._check(_LIB.csd_profile(self._h, int(enable)))

    def profile_read(self) -> dict:
        out = {}
        for i, name in enumerate(self.KERNEL_CLASSES):
            n, ms, fl = C.c_int64(), C.c_double(), C.c_double()
            self._check(_LIB.csd_profile_read(self._h, i, C.byref(n), C.byref(ms), C.byref(fl)))
            out[name] = {"launches": n.value, "ms": ms.value, "flops": fl.value}
        return out

    def close(self):
        for h in list(self._heads):
            h.close()
        if self._h:
            _LIB.csd_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- calls, named as in the C ABI ------------------------------------------------------
    def csd_draft_denoise(self, head: "Head", sched: Schedule, R, cfg, cfg_scale, z, x_T, eps, x0, mu1, x1=None):
        self._check(_LIB.csd_draft_denoise(self._h, head._h, C.byref(sched.c), R, int(cfg), cfg_scale,
                                           _ptr(z), _ptr(x_T), _ptr(eps), _ptr(x0), _ptr(mu1), _ptr(x1)))

    def csd_draft_denoise_static(self, head: "Head", sched: Schedule, R, cfg, cfg_scale, z, x_T, eps, x0, mu1, x1=None):
        """csd_draft_denoise with its intermediates in the library's built-in 8 MiB device array: no allocation."""
        self._check(_LIB.csd_draft_denoise_static(self._h, head._h, C.byref(sched.c), R, int(cfg), cfg_scale,
                                                  _ptr(z), _ptr(x_T), _ptr(eps), _ptr(x0), _ptr(mu1), _ptr(x1)))

    def csd_verify(self, head_p: "Head", sched_p: Schedule, sched_q: Schedule, B, gamma, cfg, cfg_scale,
                   z_p, x_T, eps, x0_q, mu1_q, u, logratio, n_accept, accept_mask, mu1_p):
        self._check(_LIB.csd_verify(self._h, head_p._h, C.byref(sched_p.c), C.byref(sched_q.c), B, gamma, int(cfg),
                                    cfg_scale, _ptr(z_p), _ptr(x_T), _ptr(eps), _ptr(x0_q), _ptr(mu1_q), _ptr(u),
                                    _ptr(logratio), _ptr(n_accept), _ptr(accept_mask), _ptr(mu1_p)))

    def csd_draft_denoise_traj(self, head: "Head", sched: Schedule, R, cfg, cfg_scale, z, x_T, eps, traj_x, traj_mu):
        self._check(_LIB.csd_draft_denoise_traj(self._h, head._h, C.byref(sched.c), R, int(cfg), cfg_scale,
                                                _ptr(z), _ptr(x_T), _ptr(eps), _ptr(traj_x), _ptr(traj_mu)))

    def csd_verify_single_path(self, head_p: "Head", sched_p: Schedule, sched_q: Schedule, B, gamma, cfg, cfg_scale,
                               z_p, traj_x, traj_mu_q, u, steps_per_pass, logratio, n_accept, accept_mask=None,
                               mu_p_traj=None):
        self._check(_LIB.csd_verify_single_path(self._h, head_p._h, C.byref(sched_p.c), C.byref(sched_q.c), B, gamma,
                                                int(cfg), cfg_scale, _ptr(z_p), _ptr(traj_x), _ptr(traj_mu_q),
                                                _ptr(u), int(steps_per_pass), _ptr(logratio), _ptr(n_accept),
                                                _ptr(accept_mask), _ptr(mu_p_traj)))

    def csd_verify_unaligned(self, head_p: "Head", sched_p: Schedule, sched_q: Schedule, B, gamma, cfg, cfg_scale,
                             z_p, x_T, eps_p, eps_q, x0_q, mu1_q, u, logratio, n_accept, accept_mask, mu1_p):
        self._check(_LIB.csd_verify_unaligned(self._h, head_p._h, C.byref(sched_p.c), C.byref(sched_q.c), B, gamma,
                                              int(cfg), cfg_scale, _ptr(z_p), _ptr(x_T), _ptr(eps_p), _ptr(eps_q),
                                              _ptr(x0_q), _ptr(mu1_q), _ptr(u), _ptr(logratio), _ptr(n_accept),
                                              _ptr(accept_mask), _ptr(mu1_p)))

    def csd_bonus_token(self, head_p: "Head", sched_p: Schedule, B, gamma, cfg, cfg_scale, z_next, x_T_next, eps_next,
                        n_accept, x_bonus, taken=None):
        self._check(_LIB.csd_bonus_token(self._h, head_p._h, C.byref(sched_p.c), B, gamma, int(cfg), cfg_scale,
                                         _ptr(z_next), _ptr(x_T_next), _ptr(eps_next), _ptr(n_accept), _ptr(x_bonus),
                                         _ptr(taken)))

    def csd_verify_bonus(self, head_p: "Head", sched_p: Schedule, sched_q: Schedule, B, gamma, cfg, cfg_scale, z_p, x_T,
                         eps, x0_q, mu1_q, u, z_next, x_T_next, eps_next, logratio, n_accept, accept_mask, mu1_p,
                         x_bonus, taken=None):
        self._check(_LIB.csd_verify_bonus(self._h, head_p._h, C.byref(sched_p.c), C.byref(sched_q.c), B, gamma, int(cfg),
                                          cfg_scale, *[_ptr(t) for t in (z_p, x_T, eps, x0_q, mu1_q, u, z_next, x_T_next,
                                                                         eps_next, logratio, n_accept, accept_mask, mu1_p,
                                                                         x_bonus, taken)]))

    def csd_round_bonus(self, head_q, head_p, sched_q, sched_p, B, gamma, cfg, cfg_scale, cap, z_q, z_p, x_T, eps, u, xi,
                        v, z_next, x_T_next, eps_next, x0, mu1_q, mu1_p, logratio, n_accept, accept_mask, x_new, n_prop,
                        flags, cap_hits, x_bonus, taken=None):
        self._check(_LIB.csd_round_bonus(self._h, head_q._h, head_p._h, C.byref(sched_q.c), C.byref(sched_p.c), B, gamma,
                                         int(cfg), cfg_scale, cap,
                                         *[_ptr(t) for t in (z_q, z_p, x_T, eps, u, xi, v, z_next, x_T_next, eps_next, x0,
                                                             mu1_q, mu1_p, logratio, n_accept, accept_mask, x_new, n_prop,
                                                             flags, cap_hits, x_bonus, taken)]))

    def csd_accept_scan(self, B, gamma, Cdim, log_sigma, sigma1_p, sigma1_q, x0_q, mu1_q, mu1_p, u, logratio,
                        n_accept, accept_mask=None):
        self._check(_LIB.csd_accept_scan(self._h, B, gamma, Cdim, log_sigma, sigma1_p, sigma1_q, _ptr(x0_q),
                                         _ptr(mu1_q), _ptr(mu1_p), _ptr(u), _ptr(logratio), _ptr(n_accept),
                                         _ptr(accept_mask)))

    def csd_resample(self, B, gamma, Cdim, cap, log_sigma, sigma1_p, sigma1_q, n_accept, mu1_p, mu1_q, xi, v,
                     x_new, n_prop, flags, cap_hits):
        self._check(_LIB.csd_resample(self._h, B, gamma, Cdim, cap, log_sigma, sigma1_p, sigma1_q, _ptr(n_accept),
                                      _ptr(mu1_p), _ptr(mu1_q), _ptr(xi), _ptr(v), _ptr(x_new), _ptr(n_prop),
                                      _ptr(flags), _ptr(cap_hits)))

    def csd_draft_denoise_lv(self, head: "Head", sched: ScheduleLV, R, cfg, cfg_scale, z, x_T, eps, x0, mu1, lv1,
                             half_logdet, x1=None):
        self._check(_LIB.csd_draft_denoise_lv(self._h, head._h, C.byref(sched.c), R, int(cfg), cfg_scale,
                                              *[_ptr(t) for t in (z, x_T, eps, x0, mu1, lv1, half_logdet, x1)]))

    def csd_verify_lv(self, head_p: "Head", sched_p: ScheduleLV, B, gamma, cfg, cfg_scale, z_p, x_T, eps, x0_q, mu1_q,
                      lv1_q, half_logdet_q, u, logratio, n_accept, accept_mask, mu1_p, lv1_p, half_logdet_p,
                      log_sigma_rows):
        self._check(_LIB.csd_verify_lv(self._h, head_p._h, C.byref(sched_p.c), B, gamma, int(cfg), cfg_scale,
                                       *[_ptr(t) for t in (z_p, x_T, eps, x0_q, mu1_q, lv1_q, half_logdet_q, u, logratio,
                                                           n_accept, accept_mask, mu1_p, lv1_p, half_logdet_p,
                                                           log_sigma_rows)]))

    def csd_resample_lv(self, B, gamma, Cdim, cap, log_sigma_rows, n_accept, mu1_p, lv1_p, mu1_q, lv1_q, xi, v, x_new,
                        n_prop, flags, cap_hits):
        self._check(_LIB.csd_resample_lv(self._h, B, gamma, Cdim, cap,
                                         *[_ptr(t) for t in (log_sigma_rows, n_accept, mu1_p, lv1_p, mu1_q, lv1_q, xi, v,
                                                             x_new, n_prop, flags, cap_hits)]))

    def csd_round_lv(self, head_q, head_p, sched_q: ScheduleLV, sched_p: ScheduleLV, B, gamma, cfg, cfg_scale, cap,
                     z_q, z_p, x_T, eps, u, xi, v, x0, mu1_q, lv1_q, half_logdet_q, mu1_p, lv1_p, half_logdet_p,
                     log_sigma_rows, logratio, n_accept, accept_mask, x_new, n_prop, flags, cap_hits):
        self._check(_LIB.csd_round_lv(self._h, head_q._h, head_p._h, C.byref(sched_q.c), C.byref(sched_p.c), B, gamma,
                                      int(cfg), cfg_scale, cap,
                                      *[_ptr(t) for t in (z_q, z_p, x_T, eps, u, xi, v, x0, mu1_q, lv1_q, half_logdet_q,
                                                          mu1_p, lv1_p, half_logdet_p, log_sigma_rows, logratio, n_accept,
                                                          accept_mask, x_new, n_prop, flags, cap_hits)]))

    @staticmethod
    def _gmm(m):
        """m: (logw [rows,K], mu [rows,K,C], log_sigma [rows,K,C]) device tensors."""
        logw, mu, ls = m
        return _Gmm(int(logw.shape[1]), _ptr(logw), _ptr(mu), _ptr(ls))

    def csd_gmm_draft_sample(self, R, Cdim, q, u_comp, noise, x, comp=None):
        g = self._gmm(q)
        self._check(_LIB.csd_gmm_draft_sample(self._h, R, Cdim, C.byref(g), _ptr(u_comp), _ptr(noise), _ptr(x), _ptr(comp)))

    def csd_gmm_verify(self, B, gamma, Cdim, q, p, x, u, logratio, n_accept, accept_mask=None):
        gq, gp_ = self._gmm(q), self._gmm(p)
        self._check(_LIB.csd_gmm_verify(self._h, B, gamma, Cdim, C.byref(gq), C.byref(gp_), _ptr(x), _ptr(u), _ptr(logratio),
                                        _ptr(n_accept), _ptr(accept_mask)))

    def csd_gmm_resample(self, B, gamma, Cdim, cap, q, p, n_accept, w, xi, v, x_new, n_prop, flags, cap_hits):
        gq, gp_ = self._gmm(q), self._gmm(p)
        self._check(_LIB.csd_gmm_resample(self._h, B, gamma, Cdim, cap, C.byref(gq), C.byref(gp_), _ptr(n_accept), _ptr(w),
                                          _ptr(xi), _ptr(v), _ptr(x_new), _ptr(n_prop), _ptr(flags), _ptr(cap_hits)))

    def _round(self, fn, head_q, head_p, sched_q, sched_p, B, gamma, cfg, cfg_scale, cap, z_q, z_p, x_T, eps, u,
               xi, v, x0, mu1_q, mu1_p, logratio, n_accept, accept_mask, x_new, n_prop, flags, cap_hits):
        self._check(fn(self._h, head_q._h, head_p._h, C.byref(sched_q.c), C.byref(sched_p.c), B, gamma, int(cfg),
                       cfg_scale, cap, *[_ptr(t) for t in (z_q, z_p, x_T, eps, u, xi, v, x0, mu1_q, mu1_p, logratio,
                                                           n_accept, accept_mask, x_new, n_prop, flags, cap_hits)]))

    def csd_round(self, *args):
        self._round(_LIB.csd_round, *args)

    def csd_round_host(self, *args):
        self._round(_LIB.csd_round_host, *args)


class Head:
    def __init__(self, ctx: Context, weights: Dict[str, np.ndarray], operand: str, var_out: bool = False):
        """operand: "f32", "bf16" or "f16" = the GEMM operand format; var_out: the head has 2C outputs, the second
        half being the variance parameter (see csd_head_desc)."""
        Wd, Dz = weights["Wz"].shape
        Cdim = weights["Wout"].shape[0] // (2 if var_out else 1)
        L = weights["W1"].shape[0]
        F = weights["Wt1"].shape[1]
        self.desc = _HeadDesc(Cdim, Wd, L, Dz, F, DTYPES[operand], int(var_out))
        keep = {k: np.ascontiguousarray(weights[k], dtype=np.float32) for k in WEIGHT_FIELDS}
        hw = _HeadWeights(*[keep[k].ctypes.data_as(_c_float_p) for k in WEIGHT_FIELDS])
        self._h = C.c_void_p()
        self.ctx = ctx
        rc = _LIB.csd_head_create(ctx._h, C.byref(self.desc), C.byref(hw), C.byref(self._h))
        ctx._check(rc)
        ctx._heads.append(self)

    def close(self):
        if self._h:
            _LIB.csd_head_destroy(self._h)
            self._h = C.c_void_p()
            if self in self.ctx._heads:
                self.ctx._heads.remove(self)
