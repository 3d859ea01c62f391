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
    warm_start: bool = False
    time_buffer: bool = False
    oversample: int = 0

    @property
    def n_rounds(self) -> int:
        return self.rounds if self.rounds is not None else self.wl.rounds

    @property
    def n_H(self) -> int:
        return self.H if self.H is not None else self.wl.H


def _np_state(x) -> np.ndarray:
    return x.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def _moments(x, orc: lo.LordoOracle, i: int) -> np.ndarray:
    """Moments of matrix i as the oracle holds them: the CUDA path keeps [K][r][.] for either side, the
    oracle's right-side moments are [K][rows][r]."""
    a = _np_state(x)
    return np.swapaxes(a, 1, 2) if orc.side(i) == 1 else a


def f32(x: float) -> float:
    """The value a C `float` argument carries: both sides are fed the same fp32 hyper-parameters."""
    return float(np.float32(x))


def run_oracle(spec: RunSpec, grads_fn=None) -> lo.LordoOracle:
    wl = spec.wl
    orc = make_oracle(spec)
    fn = grads_fn or (lambda rnd, h: synth.gradients(wl, spec.seed, rnd, h))
    lo.run_rounds(orc, fn, spec.n_rounds, f32(spec.lr), f32(spec.beta1), f32(spec.omega), spec.form, refresh=spec.refresh)
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
                       check_mode=spec.check_mode, warm_start=int(spec.warm_start), time_buffer=int(spec.time_buffer), oversample=spec.oversample,
                       sides=wl.sides)


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


def make_oracle(spec: RunSpec) -> lo.LordoOracle:
    wl = spec.wl
    cfg = lo.OracleConfig(mats=wl.mats, K=wl.K, H=spec.n_H, variant=spec.variant, error_feedback=spec.error_feedback,
                          beta2=f32(spec.beta2), eps=f32(spec.eps), clip_rho=f32(wl.clip_rho), clip_scope=spec.clip_scope,
                          sync_u=spec.sync_u, sync_v=spec.sync_v, outer=spec.outer, outer_lr=f32(spec.outer_lr),
                          outer_momentum=f32(spec.outer_momentum), power_iters=wl.power_iters, seed=spec.seed,
                          w_dtype=wl.w_dtype, e_dtype=wl.e_dtype, state_dtype="f32", warm_start=spec.warm_start, time_buffer=spec.time_buffer, oversample=spec.oversample,
                          sides=wl.sides)
    return lo.LordoOracle(cfg, synth.init_weights(wl, spec.seed))


def sync_oracle_from_gpu(opt, orc: lo.LordoOracle) -> None:
    """Overwrites every state array of the oracle with the CUDA path's current state."""
    for i in range(len(orc.cfg.mats)):
        orc.W[i] = _np_state(opt.W[i])
        if opt.E[i] is not None:
            orc.E[i] = _np_state(opt.E[i])
        orc.P[i] = _np_state(opt.P[i])
        orc.u[i] = _moments(opt.u[i], orc, i)
        orc.v[i] = _moments(opt.v[i], orc, i)
        orc.X0[i] = _np_state(opt.X0[i])
        orc.Delta[i] = _np_state(opt.Delta[i])
        if opt.B[i] is not None:
            orc.B[i] = _np_state(opt.B[i])


def range_finder_bf16_rhs(S: np.ndarray, Omega: Optional[np.ndarray], P_start: Optional[np.ndarray], q: int) -> np.ndarray:
    """The oracle's range finder (same steps, same Householder QR, fp64) with the right-hand side of every
    product after the first rounded to bf16 before it is multiplied, which is the one thing the tensor-core
    refresh does differently from the plain definition (the integer sketch Omega is exact in bf16).
    Omega given: P' = qr(S Omega), then q iterations; Omega None: q iterations from P_start (warm start)."""
    P = lo.householder_qr_q(S @ Omega) if Omega is not None else np.asarray(P_start, dtype=np.float64)
    for _ in range(q):
        Z = lo.householder_qr_q(S.T @ lo.round_bf16(P))
        P = lo.householder_qr_q(S @ lo.round_bf16(Z))
    return P


def run_lockstep_refresh(spec: RunSpec, rounded_signal: bool = False, inject_delta=None):
    """Runs both sides through the whole schedule; before every subspace refresh the oracle is given
    the CUDA path's state, so that each refresh is compared on identical inputs (the signal of a
    refresh is itself the product of many rounding-sensitive steps). Returns the worst metrics seen
    directly after a refresh.

    Besides the state comparison, every refresh that rotates is checked on the CUDA path's own new
    basis: `rot_u`, `rot_v` compare its rotated moments with the oracle's rotation lines applied to
    the pre-refresh moments, the pre-refresh basis and the basis the CUDA path itself returned, so
    that they measure the rotation alone, whatever the two range finders disagree on.

    rounded_signal: the oracle's range finder is fed the signal rounded to bf16, which is what the
    tensor-core sketch of the CUDA path multiplies (Global: bf16(Delta); Local: bf16 of the fp32
    value c*G + E), so that `P_angle` shows what the two sides do differently with the same signal.
    `P_angle_bf16rhs` is then the angle to range_finder_bf16_rhs of that signal: the oracle's steps in
    the operand precision of the tensor-core products.

    inject_delta(round, matrix) -> [m, n] array: Global rule only; the pseudo-gradient both sides refresh
    from is replaced by this array after the synchronisation (Delta is a caller-owned buffer), so that
    the range finder can be tested on a signal of chosen spectrum."""
    wl = spec.wl
    opt, orc = make_gpu(spec), make_oracle(spec)
    lr, b1, om = f32(spec.lr), f32(spec.beta1), f32(spec.omega)
    worst: Dict[str, float] = {}

    def before_refresh():
        torch.cuda.synchronize()
        sync_oracle_from_gpu(opt, orc)
        return {"P": [p.copy() for p in orc.P], "u": [x.copy() for x in orc.u], "v": [x.copy() for x in orc.v], "s": orc.s,
                "refreshes": orc.refreshes}

    def after_refresh(pre, signals=None):
        torch.cuda.synchronize()
        st = compare_states(opt, orc)
        for k in ("P_angle", "P_orth", "u", "v"):
            worst[k] = max(worst.get(k, 0.0), st[k])
        if rounded_signal and signals is not None and spec.oversample == 0:
            q = max(wl.power_iters, 1) if spec.warm_start else wl.power_iters
            for i, (m, n, r) in enumerate(wl.mats):
                Pg = _np_state(opt.P[i])
                for k, S in enumerate(signals[i]):
                    if orc.side(i) == 1:
                        S = S.T
                    Om = None if spec.warm_start else lo.random_matrix(spec.seed, lo.PURPOSE_OMEGA, i, pre["refreshes"], k, S.shape[1], r)
                    Po = pre["P"][i][k] if Pg.ndim == 3 else pre["P"][i]
                    want = range_finder_bf16_rhs(S, Om, Po, q)
                    worst["P_angle_bf16rhs"] = max(worst.get("P_angle_bf16rhs", 0.0),
                                                   largest_principal_angle(want, Pg[k] if Pg.ndim == 3 else Pg))
        if pre["s"] > 0:
            for i in range(len(wl.mats)):
                Pg = _np_state(opt.P[i])
                ug, vg = _np_state(opt.u[i]), _np_state(opt.v[i])  # [K][r][.] for either side
                right = orc.side(i) == 1
                for k in range(wl.K):
                    Pn = Pg[k] if Pg.ndim == 3 else Pg
                    Po = pre["P"][i][k] if Pg.ndim == 3 else pre["P"][i]
                    u0, v0 = (pre["u"][i][k].T, pre["v"][i][k].T) if right else (pre["u"][i][k], pre["v"][i][k])
                    un, vn = lo.rotate_moments(u0, v0, Pn, Po, b1, orc.cfg.beta2, pre["s"])
                    worst["rot_u"] = max(worst.get("rot_u", 0.0), scaled_error(ug[k], un))
                    worst["rot_v"] = max(worst.get("rot_v", 0.0), scaled_error(vg[k], vn))
        if signals is not None:
            # share of the signal's energy that the CUDA path's subspace captures, relative to the
            # oracle's subspace for the same signal and sketch
            for i, per_rep in enumerate(signals):
                Pg, Po = _np_state(opt.P[i]), orc.P[i]
                if Pg.ndim == 2:
                    Pg, Po = Pg[None], Po[None]
                for k, S in enumerate(per_rep):
                    if orc.side(i) == 1:
                        S = S.T
                    ratio = float(np.sum((Pg[k].T @ S) ** 2) / max(np.sum((Po[k].T @ S) ** 2), 1e-300))
                    worst["energy"] = min(worst.get("energy", 1e9), ratio)

    def local_signals(G):
        coef = lo.clip_coefficients(G, orc.cfg.clip_rho, orc.cfg.clip_scope)
        out = []
        for i in range(len(wl.mats)):
            per = []
            for k in range(wl.K):
                S = coef[i, k] * np.asarray(G[i][k], dtype=np.float64) + (orc.E[i][k] if spec.error_feedback else 0.0)
                if rounded_signal:  # c in fp32, one fp32 rounding of c*g + e, then bf16
                    S = float(np.float32(coef[i, k])) * np.asarray(G[i][k], dtype=np.float64) + (orc.E[i][k] if spec.error_feedback else 0.0)
                    S = lo.round_bf16(S.astype(np.float32))
                per.append(S)
            out.append(per)
        return out

    for rnd in range(spec.n_rounds):
        for h in range(spec.n_H):
            G = synth.gradients(wl, spec.seed, rnd, h)
            Gd = device_grads(wl, G)
            if spec.variant == 1 and h == 0:
                pre = before_refresh()
                sig = local_signals(G)
                opt.refresh_subspace(Gd, spec.beta1)
                if rounded_signal:  # hand the oracle the rounded signal as a bare gradient
                    keep = (orc.cfg.clip_rho, orc.cfg.error_feedback)
                    orc.cfg.clip_rho, orc.cfg.error_feedback = 0.0, False
                    orc.refresh_subspace([np.stack(per) for per in sig], b1)
                    orc.cfg.clip_rho, orc.cfg.error_feedback = keep
                else:
                    orc.refresh_subspace(G, b1)
                after_refresh(pre, sig)
            opt.inner_step(Gd, spec.lr, spec.beta1, spec.omega, spec.form)
            orc.inner_step(G, lr, b1, om, spec.form)
        opt.outer_step()
        orc.outer_step()
        if spec.variant == 0:
            if inject_delta is not None:
                torch.cuda.synchronize()
                for i in range(len(wl.mats)):
                    opt.Delta[i].copy_(torch.from_numpy(np.asarray(inject_delta(rnd, i), dtype=np.float32)))
            pre = before_refresh()
            if rounded_signal:
                for i in range(len(wl.mats)):
                    orc.Delta[i] = lo.round_bf16(orc.Delta[i])
            sig = [[orc.Delta[i].copy()] for i in range(len(wl.mats))]
            opt.refresh_subspace(None, spec.beta1)
            orc.refresh_subspace(None, b1)
            after_refresh(pre, sig)
    torch.cuda.synchronize()
    return opt, orc, worst


# ----------------------------------------------------------------------------------------------
# comparison metrics
# ----------------------------------------------------------------------------------------------

def weight_error(got: np.ndarray, want: np.ndarray) -> float:
    """max_ij |a-b| / max(|b_ij|, rms(b)): the element-wise relative error, with elements smaller
    than the matrix RMS measured against the RMS. (An Adam-type update is lr * u^/(sqrt(v^)+eps)
    whatever the size of the weight it lands on, so the absolute accuracy of a trajectory is set by
    the typical weight, not by an element that happens to sit near zero.)"""
    rms = float(np.sqrt(np.mean(want ** 2)))
    den = np.maximum(np.abs(want), rms + 1e-30)
    return float(np.max(np.abs(got - want) / den))


def weight_error_strict(got: np.ndarray, want: np.ndarray) -> float:
    """The same ratio with the floor at 1e-2 * rms(b): tells a 1e-6 from a 1e-3 absolute error on
    the small weights, which the rms floor cannot."""
    rms = float(np.sqrt(np.mean(want ** 2)))
    den = np.maximum(np.abs(want), 1e-2 * rms + 1e-30)
    return float(np.max(np.abs(got - want) / den))


def frobenius_error(got: np.ndarray, want: np.ndarray) -> float:
    return float(np.linalg.norm(got - want) / (np.linalg.norm(want) + 1e-300))


def scaled_error(got: np.ndarray, want: np.ndarray) -> float:
    """max |a-b| / max|b| -- for states whose elements span many magnitudes."""
    return float(np.max(np.abs(got - want)) / (np.max(np.abs(want)) + 1e-30))


def largest_principal_angle(A: np.ndarray, B: np.ndarray) -> float:
    """Largest principal angle between span(A) and span(B) (orthonormal columns), computed from
    sin(theta_max) = ||(I - A A^T) B||_2, which stays accurate for small angles."""
    R = B - A @ (A.T @ B)
    return float(np.arcsin(min(1.0, np.linalg.norm(R, 2))))


def bf16_ulp_distance(got: np.ndarray, want: np.ndarray) -> np.ndarray:
    """|a-b| in units of the bf16 spacing at max(|b_ij|, rms(b)) (8 significant bits: the spacing at
    x is 2^(floor(log2 x) - 7)). Elements below the RMS are measured in the spacing at the RMS,
    for the reason given in weight_error."""
    rms = float(np.sqrt(np.mean(want ** 2)))
    ref = np.maximum(np.abs(want), rms + 1e-30)
    ulp = 2.0 ** (np.floor(np.log2(ref)) - 7)
    return np.abs(got - want) / ulp


def compare_states(opt, orc: lo.LordoOracle) -> Dict[str, float]:
    """Worst-case metrics over all matrices between the CUDA state and the oracle state."""
    out = {"W": 0.0, "W_strict": 0.0, "W_fro": 0.0, "E": 0.0, "u": 0.0, "v": 0.0, "X0": 0.0, "Delta": 0.0, "B": 0.0,
           "P_angle": 0.0, "P_orth": 0.0, "P_cols": 0.0}
    for i in range(len(orc.cfg.mats)):
        Wg = _np_state(opt.W[i])
        out["W"] = max(out["W"], weight_error(Wg, orc.W[i]))
        out["W_strict"] = max(out["W_strict"], weight_error_strict(Wg, orc.W[i]))
        out["W_fro"] = max(out["W_fro"], frobenius_error(Wg, orc.W[i]))
        if opt.E[i] is not None:
            out["E"] = max(out["E"], scaled_error(_np_state(opt.E[i]), orc.E[i]))
        out["u"] = max(out["u"], scaled_error(_moments(opt.u[i], orc, i), orc.u[i]))
        out["v"] = max(out["v"], scaled_error(_moments(opt.v[i], orc, i), orc.v[i]))
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
