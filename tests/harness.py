"""Drives the CUDA path and the CPU oracle over the same seeded inputs and compares their states."""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import numpy as np
import torch

from oracle import lordo_oracle as lo
from paper_2602_04396_b200 import synth

BF16_EPS = 2.0 ** -8


@dataclasses.dataclass
class RunSpec:
    wl: synth.Workload
    seed: int = 0
    variant: int = 0  # 0 Global, 1 Local
    form: int = 0
    error_feedback: bool = True
    outer: int = 0
    outer_lr: float = 0.8
    outer_momentum: float = 0.9
    lr: float = 0.004
    beta1: float = 0.9
    beta2: float = 0.999
    omega: float = 0.97
    eps: float = 1e-8
    clip_scope: int = 0
    sync_u: bool = True
    sync_v: bool = True
    refresh: bool = True
    rounds: Optional[int] = None
    H: Optional[int] = None
    check_mode: int = 1

    @property
    def n_rounds(self) -> int:
        return self.rounds if self.rounds is not None else self.wl.rounds

    @property
    def n_H(self) -> int:
        return self.H if self.H is not None else self.wl.H


def _np_state(x) -> np.ndarray:
    return x.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def run_oracle(spec: RunSpec, grads_fn=None) -> lo.LordoOracle:
    wl = spec.wl
    cfg = lo.OracleConfig(mats=wl.mats, K=wl.K, H=spec.n_H, variant=spec.variant, error_feedback=spec.error_feedback,
                          beta2=spec.beta2, eps=spec.eps, clip_rho=wl.clip_rho, clip_scope=spec.clip_scope,
                          sync_u=spec.sync_u, sync_v=spec.sync_v, outer=spec.outer, outer_lr=spec.outer_lr,
                          outer_momentum=spec.outer_momentum, power_iters=wl.power_iters, seed=spec.seed,
                          w_dtype=wl.w_dtype, e_dtype=wl.e_dtype, state_dtype="f32")
    orc = lo.LordoOracle(cfg, synth.init_weights(wl, spec.seed))
    fn = grads_fn or (lambda rnd, h: synth.gradients(wl, spec.seed, rnd, h))
    lo.run_rounds(orc, fn, spec.n_rounds, spec.lr, spec.beta1, spec.omega, spec.form, refresh=spec.refresh)
    return orc


def make_gpu(spec: RunSpec):
    from paper_2602_04396_b200 import lordo
    wl = spec.wl
    W0 = [torch.from_numpy(w).to(synth.torch_dtype(wl.w_dtype)) for w in synth.init_weights(wl, spec.seed)]
    return lordo.Lordo(wl.mats, wl.K, spec.n_H, W0, g_dtype=synth.torch_dtype(wl.g_dtype),
                       e_dtype=synth.torch_dtype(wl.e_dtype), variant=spec.variant, error_feedback=spec.error_feedback,
                       beta2=spec.beta2, eps=spec.eps, clip_rho=wl.clip_rho, clip_scope=spec.clip_scope,
                       sync_u=spec.sync_u, sync_v=spec.sync_v, outer=spec.outer, outer_lr=spec.outer_lr,
                       outer_momentum=spec.outer_momentum, power_iters=wl.power_iters, seed=spec.seed,
                       check_mode=spec.check_mode)


def device_grads(wl: synth.Workload, G: List[np.ndarray]) -> List[torch.Tensor]:
    return [torch.from_numpy(g).to(synth.torch_dtype(wl.g_dtype)).cuda().contiguous() for g in G]


def run_gpu(spec: RunSpec, grads_fn=None):
    wl = spec.wl
    opt = make_gpu(spec)
    fn = grads_fn or (lambda rnd, h: synth.gradients(wl, spec.seed, rnd, h))
    for rnd in range(spec.n_rounds):
        for h in range(spec.n_H):
            G = device_grads(wl, fn(rnd, h))
            if spec.refresh and spec.variant == 1 and h == 0:
                opt.refresh_subspace(G, spec.beta1)
            opt.inner_step(G, spec.lr, spec.beta1, spec.omega, spec.form)
        opt.outer_step()
        if spec.refresh and spec.variant == 0:
            opt.refresh_subspace(None, spec.beta1)
    torch.cuda.synchronize()
    return opt


# ----------------------------------------------------------------------------------------------
# comparison metrics
# ----------------------------------------------------------------------------------------------

def weight_error(got: np.ndarray, want: np.ndarray) -> float:
    """max_ij |a-b| / max(|b_ij|, 1e-3 rms(b)): the element-wise relative error with a floor that
    keeps elements near zero from dominating."""
    rms = float(np.sqrt(np.mean(want ** 2)))
    den = np.maximum(np.abs(want), 1e-3 * rms + 1e-30)
    return float(np.max(np.abs(got - want) / den))


def scaled_error(got: np.ndarray, want: np.ndarray) -> float:
    """max |a-b| / max|b| -- for states whose elements span many magnitudes."""
    return float(np.max(np.abs(got - want)) / (np.max(np.abs(want)) + 1e-30))


def largest_principal_angle(A: np.ndarray, B: np.ndarray) -> float:
    """Largest principal angle between span(A) and span(B) (orthonormal columns), computed from
    sin(theta_max) = ||(I - A A^T) B||_2, which stays accurate for small angles."""
    R = B - A @ (A.T @ B)
    return float(np.arcsin(min(1.0, np.linalg.norm(R, 2))))


def bf16_ulp_distance(got: np.ndarray, want: np.ndarray) -> np.ndarray:
    """Distance in bf16 units of least precision between two arrays of bf16-representable values."""
    def key(x):
        b = x.astype(np.float32).view(np.uint32).astype(np.int64) >> 16
        return np.where(b & 0x8000, 0x8000 - b, b)  # monotone integer key
    return np.abs(key(got) - key(want))


def compare_states(opt, orc: lo.LordoOracle) -> Dict[str, float]:
    """Worst-case metrics over all matrices between the CUDA state and the oracle state."""
    out = {"W": 0.0, "E": 0.0, "u": 0.0, "v": 0.0, "X0": 0.0, "Delta": 0.0, "B": 0.0, "P_angle": 0.0, "P_orth": 0.0,
           "P_cols": 0.0}
    for i in range(len(orc.cfg.mats)):
        out["W"] = max(out["W"], weight_error(_np_state(opt.W[i]), orc.W[i]))
        if opt.E[i] is not None:
            out["E"] = max(out["E"], scaled_error(_np_state(opt.E[i]), orc.E[i]))
        out["u"] = max(out["u"], scaled_error(_np_state(opt.u[i]), orc.u[i]))
        out["v"] = max(out["v"], scaled_error(_np_state(opt.v[i]), orc.v[i]))
        out["X0"] = max(out["X0"], weight_error(_np_state(opt.X0[i]), orc.X0[i]))
        out["Delta"] = max(out["Delta"], scaled_error(_np_state(opt.Delta[i]), orc.Delta[i]))
        if opt.B[i] is not None:
            out["B"] = max(out["B"], scaled_error(_np_state(opt.B[i]), orc.B[i]))
        Pg, Po = _np_state(opt.P[i]), orc.P[i]
        if Pg.ndim == 2:
            Pg, Po = Pg[None], Po[None]
        for k in range(Pg.shape[0]):
            out["P_angle"] = max(out["P_angle"], largest_principal_angle(Po[k], Pg[k]))
            out["P_orth"] = max(out["P_orth"], float(np.abs(Pg[k].T @ Pg[k] - np.eye(Pg.shape[2])).max()))
            out["P_cols"] = max(out["P_cols"], float(np.abs(Pg[k] - Po[k]).max()))
    return out
