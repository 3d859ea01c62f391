"""Seeded synthetic inputs for the LoRDO optimizer hot path.

This module only *produces inputs* (layer shapes, initial weights, gradients). It holds none of
the method's arithmetic, so that the CPU oracle and the CUDA path can both be fed from it without
sharing any code of the method itself.

The paper trains decoder LMs on a text mixture (Sec. "Experimental Framework", Table "Model
architecture"); no dataset is needed for the optimizer path, so synthetic gradients with the
shapes of the paper's layers stand in for back-propagated ones:

* weights      ~ N(0, 0.02^2)                     (Table "Model architecture": init sigma 0.02)
* ``gauss``    : G ~ N(0,1) i.i.d. per replica and step
* ``lowrank``  : G = U V^T / sqrt(k) + 0.1 N(0,1) with Gaussian factors U (m x k), V (n x k),
                 k = 32, redrawn once per round and shared by the replicas (the paper splits the
                 data IID across workers), noise redrawn per replica and step
* ``student``  : heavy-tailed Student-t (nu = 3) entries scaled to unit RMS per matrix

Every stream is addressed by (seed, tag, matrix, replica, round, step) so that any single gradient
can be regenerated in isolation.
"""
from __future__ import annotations

import dataclasses
from typing import List, Sequence, Tuple

import numpy as np
import torch

F32 = "f32"
BF16 = "bf16"

_TAG_W0, _TAG_NOISE, _TAG_U, _TAG_V, _TAG_T = 1, 2, 3, 4, 5


@dataclasses.dataclass(frozen=True)
class Workload:
    """One benchmark / parity configuration (shapes and schedule only)."""

    name: str
    mats: Tuple[Tuple[int, int, int], ...]  # (m, n, r) per weight matrix, W is m x n, P is m x r
    K: int  # simulated workers (paper: M)
    H: int  # inner steps per round (paper: K_x)
    rounds: int
    w_dtype: str = F32
    g_dtype: str = F32
    e_dtype: str = F32
    grad: str = "gauss"  # gauss | lowrank | student
    power_iters: int = 0
    refresh_every_step: bool = False
    clip_rho: float = 1.0
    signal_rank: int = 32
    noise: float = 0.1
    sides: Tuple[int, ...] | None = None  # per matrix: 1 = the basis is applied from the right (default: all from the left)

    @property
    def weights(self) -> int:
        return sum(m * n for m, n, _ in self.mats)

    @property
    def weight_replicas(self) -> int:
        return self.weights * self.K


def _decoder_stack(layers: int, d: int, ffn: int, r: int) -> Tuple[Tuple[int, int, int], ...]:
    per_layer = [(d, d, r)] * 4 + [(d, ffn, r)] * 2 + [(ffn, d, r)]
    return tuple(per_layer * layers)


def config(index: int, r: int | None = None) -> Workload:
    """The five configurations of the build contract, by 1-based index."""
    if index == 1:
        return Workload("cfg1_256x256_r16", ((256, 256, 16),), K=2, H=4, rounds=3, grad="gauss", clip_rho=1.0)
    if index == 2:
        return Workload("cfg2_2048x2048_r128", ((2048, 2048, 128),), K=4, H=32, rounds=4, grad="lowrank",
                        clip_rho=1.0)
    if index == 3:
        rr = 128 if r is None else r
        return Workload(f"cfg3_125M_r{rr}", _decoder_stack(12, 768, 3072, rr), K=8, H=64, rounds=2,
                        w_dtype=BF16, g_dtype=BF16, e_dtype=BF16, grad="lowrank", clip_rho=0.5)
    if index == 4:
        return Workload("cfg4_1B_r256", _decoder_stack(24, 2048, 5632, 256), K=8, H=128, rounds=2,
                        w_dtype=BF16, g_dtype=BF16, e_dtype=BF16, grad="lowrank", clip_rho=0.1)
    if index == 5:
        return Workload("cfg5_refresh_stress", ((4096, 11008, 512),) * 32, K=16, H=1, rounds=2,
                        w_dtype=BF16, g_dtype=BF16, e_dtype=BF16, grad="student", power_iters=2,
                        refresh_every_step=True, clip_rho=1.0)
    raise ValueError(f"no config {index}")


def scaled(wl: Workload, *, mats: Sequence[Tuple[int, int, int]] | None = None, **kw) -> Workload:
    """A copy of ``wl`` with some fields replaced (used for sampled / reduced parity cases)."""
    if mats is not None:
        kw["mats"] = tuple(tuple(x) for x in mats)
    return dataclasses.replace(wl, **kw)


# ----------------------------------------------------------------------------------------------
# host generators (numpy): bit-reproducible, used by the parity tests for both sides
# ----------------------------------------------------------------------------------------------

def _rng(seed: int, tag: int, *ids: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([seed, tag, *[int(i) for i in ids]])))


def to_bf16_grid(x: np.ndarray) -> np.ndarray:
    """Round an fp32 array to the nearest bf16 value, returned as fp32 (input preparation only)."""
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy()


def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    x = np.asarray(x, dtype=np.float32)
    return to_bf16_grid(x) if dtype == BF16 else x


def init_weights(wl: Workload, seed: int) -> List[np.ndarray]:
    """W0 per matrix, fp32 arrays (on the bf16 grid when the workload stores bf16 weights)."""
    out = []
    for i, (m, n, _) in enumerate(wl.mats):
        w = _rng(seed, _TAG_W0, i).standard_normal((m, n), dtype=np.float32) * np.float32(0.02)
        out.append(_store(w, wl.w_dtype))
    return out


def gradient(wl: Workload, seed: int, mat: int, replica: int, rnd: int, step: int) -> np.ndarray:
    """The synthetic gradient of one matrix for one replica at (round, step); fp32 array m x n."""
    m, n, _ = wl.mats[mat]
    if wl.grad == "gauss":
        g = _rng(seed, _TAG_NOISE, mat, replica, rnd, step).standard_normal((m, n), dtype=np.float32)
    elif wl.grad == "lowrank":
        k = wl.signal_rank
        U = _rng(seed, _TAG_U, mat, rnd).standard_normal((m, k), dtype=np.float32)
        V = _rng(seed, _TAG_V, mat, rnd).standard_normal((n, k), dtype=np.float32)
        noise = _rng(seed, _TAG_NOISE, mat, replica, rnd, step).standard_normal((m, n), dtype=np.float32)
        g = (U @ V.T) / np.float32(np.sqrt(k)) + np.float32(wl.noise) * noise
    elif wl.grad == "student":
        z = _rng(seed, _TAG_T, mat, replica, rnd, step).standard_normal((4, m, n), dtype=np.float32)
        t = z[0] / np.sqrt((z[1] ** 2 + z[2] ** 2 + z[3] ** 2) / np.float32(3.0))
        g = t / np.sqrt(np.mean(t.astype(np.float64) ** 2)).astype(np.float32)
    else:
        raise ValueError(wl.grad)
    return _store(g, wl.g_dtype)


def gradients(wl: Workload, seed: int, rnd: int, step: int) -> List[np.ndarray]:
    """All gradients of one step: list over matrices of fp32 arrays [K, m, n]."""
    return [np.stack([gradient(wl, seed, i, k, rnd, step) for k in range(wl.K)]) for i in range(len(wl.mats))]


# ----------------------------------------------------------------------------------------------
# device generators (torch, CUDA): for workloads too large to build on the host
# ----------------------------------------------------------------------------------------------

def torch_dtype(name: str) -> torch.dtype:
    return torch.bfloat16 if name == BF16 else torch.float32


def init_weights_device(wl: Workload, seed: int, device: str = "cuda") -> List[torch.Tensor]:
    gen = torch.Generator(device=device)
    out = []
    for i, (m, n, _) in enumerate(wl.mats):
        gen.manual_seed((seed * 1000003 + i) & 0x7FFFFFFF)
        w = torch.empty((m, n), device=device, dtype=torch.float32).normal_(0.0, 0.02, generator=gen)
        out.append(w.to(torch_dtype(wl.w_dtype)))
    return out


def gradients_device(wl: Workload, seed: int, rnd: int, step: int, device: str = "cuda",
                     out: List[torch.Tensor] | None = None) -> List[torch.Tensor]:
    """All gradients of one step on the device: list over matrices of tensors [K, m, n] in g_dtype."""
    gen = torch.Generator(device=device)
    res = []
    for i, (m, n, _) in enumerate(wl.mats):
        gen.manual_seed((((seed * 1009 + i) * 1013 + rnd) * 1019 + step) & 0x7FFFFFFFFFFF)
        dst = out[i] if out is not None else torch.empty((wl.K, m, n), device=device, dtype=torch_dtype(wl.g_dtype))
        if wl.grad == "gauss":
            dst.copy_(torch.empty((wl.K, m, n), device=device).normal_(generator=gen))
        elif wl.grad == "lowrank":
            k = wl.signal_rank
            U = torch.empty((m, k), device=device).normal_(generator=gen)
            V = torch.empty((n, k), device=device).normal_(generator=gen)
            sig = (U @ V.T) / (k ** 0.5)
            for rep in range(wl.K):
                dst[rep].copy_(sig + wl.noise * torch.empty((m, n), device=device).normal_(generator=gen))
        elif wl.grad == "student":
            for rep in range(wl.K):
                z = torch.empty((4, m, n), device=device).normal_(generator=gen)
                t = z[0] / torch.sqrt((z[1] ** 2 + z[2] ** 2 + z[3] ** 2) / 3.0)
                dst[rep].copy_(t / torch.sqrt(torch.mean(t.double() ** 2)).float())
        else:
            raise ValueError(wl.grad)
        res.append(dst)
    return res
