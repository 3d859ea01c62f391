"""Thin ctypes binding of the C ABI in include/lordo.h (argument marshalling only).

PyTorch is used for device memory and streams; every step of the path runs in the library's CUDA
kernels. There is no fallback: if the shared library is missing or fails to load, importing the
symbols raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

import torch

F32, BF16 = 0, 1
GLOBAL, LOCAL = 0, 1
QHM_NONE, QHM_LOW, QHM_FULL = 0, 1, 2
OUTER_AVG, OUTER_NESTEROV = 0, 1
FLAG_NONFINITE_GRAD, FLAG_QR_BREAKDOWN = 1, 2

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "_lib", "liblordo.so")

EXPORTS = [
    "lordo_query_workspace", "lordo_init", "lordo_inner_step", "lordo_inner_step_host", "lordo_outer_step",
    "lordo_refresh_subspace", "lordo_poll_status", "lordo_get_counters", "lordo_set_counters",
    "lordo_clip_coefficients", "lordo_launch_count", "lordo_last_error", "lordo_status_string", "lordo_destroy",
    "lordo_fill_random", "lordo_profile_enable", "lordo_profile_read", "lordo_clip_coefficient_static",
    "lordo_clip_coefficient_static_max_count", "lordo_clear_status", "lordo_selftest_wait_timeout", "lordo_diagnostics", "lordo_sync_states",
]


class LordoError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: status {status} ({detail})")


class _Mat(C.Structure):
    _fields_ = [("m", C.c_int64), ("n", C.c_int64), ("r", C.c_int32), ("side", C.c_int32)]


class _Config(C.Structure):
    _fields_ = [
        ("n_mats", C.c_int32), ("mats", C.POINTER(_Mat)), ("K", C.c_int32), ("H", C.c_int32),
        ("w_dtype", C.c_int32), ("g_dtype", C.c_int32), ("e_dtype", C.c_int32), ("variant", C.c_int32),
        ("error_feedback", C.c_int32), ("beta2", C.c_float), ("eps", C.c_float), ("clip_rho", C.c_float),
        ("clip_scope", C.c_int32), ("sync_u", C.c_int32), ("sync_v", C.c_int32), ("outer", C.c_int32),
        ("outer_lr", C.c_float), ("outer_momentum", C.c_float), ("power_iters", C.c_int32), ("seed", C.c_uint64),
        ("check_mode", C.c_int32), ("warm_start", C.c_int32), ("time_buffer", C.c_int32), ("oversample", C.c_int32),
    ]


class _Buffers(C.Structure):
    _fields_ = [(name, C.POINTER(C.c_void_p)) for name in ("W", "E", "P", "u", "v", "X0", "B", "Delta")]


_lib = None


def load_library() -> C.CDLL:
    """Loads liblordo.so (built by paper_2602_04396_b200.build). Raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise FileNotFoundError(f"{_LIB_PATH} is missing: run `python -m paper_2602_04396_b200.build`")
    lib = C.CDLL(_LIB_PATH)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    lib.lordo_query_workspace.argtypes = [C.POINTER(_Config), C.POINTER(C.c_size_t)]
    lib.lordo_init.argtypes = [C.POINTER(_Config), C.POINTER(_Buffers), vp, C.c_size_t, vp, C.POINTER(vp)]
    lib.lordo_inner_step.argtypes = [vp, C.POINTER(vp), f32, f32, f32, i32, vp]
    lib.lordo_inner_step_host.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), f32, f32, f32, i32, vp, vp]
    lib.lordo_outer_step.argtypes = [vp, vp]
    lib.lordo_refresh_subspace.argtypes = [vp, C.POINTER(vp), f32, vp]
    lib.lordo_poll_status.argtypes = [vp, vp, C.POINTER(C.c_uint32)]
    lib.lordo_get_counters.argtypes = [vp, C.POINTER(i64)]
    lib.lordo_set_counters.argtypes = [vp, C.POINTER(i64)]
    lib.lordo_clip_coefficients.argtypes = [vp, C.POINTER(vp)]
    lib.lordo_launch_count.argtypes = [vp]
    lib.lordo_launch_count.restype = i64
    lib.lordo_last_error.argtypes = [vp]
    lib.lordo_last_error.restype = C.c_char_p
    lib.lordo_status_string.argtypes = [i32]
    lib.lordo_status_string.restype = C.c_char_p
    lib.lordo_destroy.argtypes = [vp]
    lib.lordo_fill_random.argtypes = [C.c_uint64, i32, i32, i64, i32, i64, i64, vp, vp]
    lib.lordo_profile_enable.argtypes = [vp, i32]
    lib.lordo_profile_read.argtypes = [vp, vp, C.POINTER(f32)]
    lib.lordo_clear_status.argtypes = [vp, vp]
    lib.lordo_sync_states.argtypes = [vp, i32, i32, vp]
    lib.lordo_diagnostics.argtypes = [vp, vp, vp, vp]
    lib.lordo_selftest_wait_timeout.argtypes = [vp, vp]
    lib.lordo_clip_coefficient_static.argtypes = [vp, i32, i64, f32, vp, vp]
    lib.lordo_clip_coefficient_static_max_count.argtypes = []
    lib.lordo_clip_coefficient_static_max_count.restype = i64
    for name in EXPORTS:
        if getattr(lib, name).restype is C.c_int:
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float32:
        return F32
    if dt == torch.bfloat16:
        return BF16
    raise ValueError(f"unsupported dtype {dt}")


def _ptr_table(tensors: Optional[Sequence[Optional[torch.Tensor]]], n: int):
    arr = (C.c_void_p * n)()
    if tensors is not None:
        for i, t in enumerate(tensors):
            arr[i] = t.data_ptr() if t is not None else None
    return arr


def _stream_handle(stream: Optional[torch.cuda.Stream]) -> C.c_void_p:
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def make_config(mats: Sequence[Tuple[int, int, int]], K: int, H: int, *, w_dtype=F32, g_dtype=F32, e_dtype=F32,
                variant=GLOBAL, error_feedback=True, beta2=0.999, eps=1e-8, clip_rho=0.0, clip_scope=0, sync_u=True,
                sync_v=True, outer=OUTER_AVG, outer_lr=1.0, outer_momentum=0.0, power_iters=0, seed=0, check_mode=1, warm_start=0, time_buffer=0, oversample=0,
                sides: Optional[Sequence[int]] = None):
    """Returns (config struct, keep-alive matrix array). sides[i] = 1 projects matrix i from the right."""
    arr = (_Mat * len(mats))()
    for i, (m, n, r) in enumerate(mats):
        arr[i] = _Mat(m, n, r, int(sides[i]) if sides is not None else 0)
    cfg = _Config(len(mats), arr, K, H, w_dtype, g_dtype, e_dtype, variant, int(error_feedback), beta2, eps, clip_rho,
                  clip_scope, int(sync_u), int(sync_v), outer, outer_lr, outer_momentum, power_iters, seed, check_mode, int(warm_start), int(time_buffer), int(oversample))
    return cfg, arr


def query_workspace(cfg: _Config) -> int:
    lib = load_library()
    out = C.c_size_t(0)
    rc = lib.lordo_query_workspace(C.byref(cfg), C.byref(out))
    if rc != 0:
        raise LordoError(rc, "lordo_query_workspace", lib.lordo_status_string(rc).decode())
    return out.value


def fill_random(seed: int, purpose: int, mat: int, index: int, replica: int, rows: int, cols: int,
                device: str = "cuda") -> torch.Tensor:
    lib = load_library()
    out = torch.empty((rows, cols), device=device, dtype=torch.float32)
    rc = lib.lordo_fill_random(seed, purpose, mat, index, replica, rows, cols, C.c_void_p(out.data_ptr()), _stream_handle(None))
    if rc != 0:
        raise LordoError(rc, "lordo_fill_random", lib.lordo_status_string(rc).decode())
    return out


def clip_coefficient_static(G: torch.Tensor, rho: float, out: torch.Tensor, stream=None) -> None:
    """Clip coefficient of one gradient tensor through lordo_clip_coefficient_static, the entry
    point that allocates no device memory. `out` is a one-element float32 CUDA tensor that the
    caller provides; nothing is allocated here either."""
    lib = load_library()
    assert G.is_cuda and G.is_contiguous() and out.is_cuda and out.dtype == torch.float32 and out.numel() == 1
    rc = lib.lordo_clip_coefficient_static(C.c_void_p(G.data_ptr()), _dtype_code(G.dtype), G.numel(), rho,
                                           C.c_void_p(out.data_ptr()), _stream_handle(stream))
    if rc != 0:
        limit = lib.lordo_clip_coefficient_static_max_count()
        raise LordoError(rc, "lordo_clip_coefficient_static",
                         f"{lib.lordo_status_string(rc).decode()}; at most {limit} elements, a multiple of 8")


class Lordo:
    """Owns the device tensors of one optimizer instance (through PyTorch) and forwards the four
    verbs to the library. W0: list of [m, n] tensors (any device) in the weight dtype."""

    def __init__(self, mats: Sequence[Tuple[int, int, int]], K: int, H: int, W0: Sequence[torch.Tensor], *,
                 device: str = "cuda", g_dtype: torch.dtype = torch.float32, e_dtype: torch.dtype = torch.float32, **kw):
        self.lib = load_library()
        self.mats = [tuple(int(x) for x in t) for t in mats]
        self.K, self.H = K, H
        self.device = torch.device(device)
        w_dt = W0[0].dtype
        self.w_dtype, self.g_dtype, self.e_dtype = w_dt, g_dtype, e_dtype
        self.variant = kw.get("variant", GLOBAL)
        self.error_feedback = bool(kw.get("error_feedback", True))
        self.outer = kw.get("outer", OUTER_AVG)
        self.sides = [int(x) for x in kw["sides"]] if kw.get("sides") is not None else [0] * len(self.mats)
        self.cfg, self._mats_keep = make_config(self.mats, K, H, w_dtype=_dtype_code(w_dt), g_dtype=_dtype_code(g_dtype),
                                                e_dtype=_dtype_code(e_dtype), **kw)
        dev = self.device
        z = lambda shape, dt=torch.float32: torch.empty(shape, device=dev, dtype=dt)
        self.W, self.E, self.P, self.u, self.v, self.X0, self.B, self.Delta = [], [], [], [], [], [], [], []
        for (m, n, r), w0, side in zip(self.mats, W0, self.sides):
            w = z((K, m, n), w_dt)
            w[0].copy_(w0.to(dev))
            self.W.append(w)
            self.E.append(z((K, m, n), e_dtype) if self.error_feedback else None)
            pm, ln = (n, m) if side else (m, n)  # rows of the basis, columns of the low-rank moments
            self.P.append(z((K, pm, r)) if self.variant == LOCAL else z((pm, r)))
            self.u.append(z((K, r, ln)))
            self.v.append(z((K, r, ln)))
            self.X0.append(z((m, n)))
            self.B.append(z((m, n)) if self.outer == OUTER_NESTEROV else None)
            self.Delta.append(z((m, n)))
        n_mats = len(self.mats)
        self._tables = {
            "W": _ptr_table(self.W, n_mats), "E": _ptr_table(self.E, n_mats) if self.error_feedback else None,
            "P": _ptr_table(self.P, n_mats), "u": _ptr_table(self.u, n_mats), "v": _ptr_table(self.v, n_mats),
            "X0": _ptr_table(self.X0, n_mats), "B": _ptr_table(self.B, n_mats) if self.outer == OUTER_NESTEROV else None,
            "Delta": _ptr_table(self.Delta, n_mats),
        }
        bufs = _Buffers(*[C.cast(self._tables[k], C.POINTER(C.c_void_p)) if self._tables[k] is not None else None
                          for k in ("W", "E", "P", "u", "v", "X0", "B", "Delta")])
        self.workspace_bytes = query_workspace(self.cfg)
        self.workspace = torch.empty(self.workspace_bytes + 256, device=dev, dtype=torch.uint8)
        base = (self.workspace.data_ptr() + 255) & ~255
        self._ctx = C.c_void_p(None)
        with torch.cuda.device(dev):
            rc = self.lib.lordo_init(C.byref(self.cfg), C.byref(bufs), C.c_void_p(base), self.workspace_bytes,
                                     _stream_handle(None), C.byref(self._ctx))
        if rc != 0:
            raise LordoError(rc, "lordo_init", self.lib.lordo_status_string(rc).decode())
        self._G_keep = None

    # -- helpers -----------------------------------------------------------------------------
    def _check(self, rc: int, where: str):
        if rc != 0:
            raise LordoError(rc, where, self.lib.lordo_last_error(self._ctx).decode())

    def _g_table(self, G: Sequence[torch.Tensor]):
        assert len(G) == len(self.mats)
        for g, (m, n, _) in zip(G, self.mats):
            assert g.is_contiguous() and tuple(g.shape) == (self.K, m, n) and g.dtype == self.g_dtype, (g.shape, g.dtype)
        tab = _ptr_table(G, len(G))
        self._G_keep = (tab, list(G))
        return C.cast(tab, C.POINTER(C.c_void_p))

    # -- the verbs ---------------------------------------------------------------------------
    def inner_step(self, G: Sequence[torch.Tensor], lr: float, beta1: float, omega: float, form: int, stream=None):
        self._check(self.lib.lordo_inner_step(self._ctx, self._g_table(G), lr, beta1, omega, form, _stream_handle(stream)),
                    "lordo_inner_step")

    def inner_step_host(self, G_host: Sequence[torch.Tensor], G_stage: Sequence[torch.Tensor], lr: float, beta1: float,
                        omega: float, form: int, clip_out: Optional[torch.Tensor] = None, stream=None):
        """G_host: host tensors ([K, m, n], pinned for full speed); G_stage: device staging tensors."""
        n = len(self.mats)
        host_tab = _ptr_table(G_host, n)
        stage_tab = _ptr_table(G_stage, n)
        self._G_keep = (host_tab, stage_tab, list(G_host), list(G_stage))
        out_ptr = C.c_void_p(clip_out.data_ptr()) if clip_out is not None else None
        self._check(self.lib.lordo_inner_step_host(self._ctx, C.cast(host_tab, C.POINTER(C.c_void_p)),
                                                   C.cast(stage_tab, C.POINTER(C.c_void_p)), lr, beta1, omega, form, out_ptr,
                                                   _stream_handle(stream)), "lordo_inner_step_host")

    def outer_step(self, stream=None):
        self._check(self.lib.lordo_outer_step(self._ctx, _stream_handle(stream)), "lordo_outer_step")

    def refresh_subspace(self, G: Optional[Sequence[torch.Tensor]] = None, beta1: float = 0.9, stream=None):
        tab = self._g_table(G) if G is not None else None
        self._check(self.lib.lordo_refresh_subspace(self._ctx, tab, beta1, _stream_handle(stream)), "lordo_refresh_subspace")

    def poll_status(self, stream=None) -> int:
        flags = C.c_uint32(0)
        rc = self.lib.lordo_poll_status(self._ctx, _stream_handle(stream), C.byref(flags))
        if rc not in (0, 7):
            self._check(rc, "lordo_poll_status")
        return flags.value

    def diagnostics(self, stream=None):
        """(mssv [number of projection matrices], e_norm [n_mats, K] or None) as device tensors."""
        nproj = len(self.mats) * (self.K if self.variant == LOCAL else 1)
        mssv = torch.empty(nproj, device=self.device, dtype=torch.float32)
        en = torch.empty((len(self.mats), self.K), device=self.device, dtype=torch.float32) if self.error_feedback else None
        self._check(self.lib.lordo_diagnostics(self._ctx, C.c_void_p(mssv.data_ptr()), C.c_void_p(en.data_ptr()) if en is not None else None,
                                               _stream_handle(stream)), "lordo_diagnostics")
        return mssv, en

    def sync_states(self, sync_u: bool, sync_v: bool, stream=None):
        self._check(self.lib.lordo_sync_states(self._ctx, int(sync_u), int(sync_v), _stream_handle(stream)), "lordo_sync_states")

    def clear_status(self, stream=None):
        self._check(self.lib.lordo_clear_status(self._ctx, _stream_handle(stream)), "lordo_clear_status")

    def selftest_wait_timeout(self, stream=None):
        self._check(self.lib.lordo_selftest_wait_timeout(self._ctx, _stream_handle(stream)), "lordo_selftest_wait_timeout")

    def counters(self) -> List[int]:
        out = (C.c_int64 * 4)()
        self._check(self.lib.lordo_get_counters(self._ctx, out), "lordo_get_counters")
        return list(out)

    def set_counters(self, values: Sequence[int]):
        arr = (C.c_int64 * 4)(*values)
        self._check(self.lib.lordo_set_counters(self._ctx, arr), "lordo_set_counters")

    def clip_coefficients(self) -> torch.Tensor:
        """[n_mats, K] clip coefficients of the last inner step (copied out of the workspace)."""
        ptr = C.c_void_p(None)
        self._check(self.lib.lordo_clip_coefficients(self._ctx, C.byref(ptr)), "lordo_clip_coefficients")
        off = ptr.value - self.workspace.data_ptr()
        n = len(self.mats) * self.K
        return self.workspace[off:off + 4 * n].view(torch.float32).view(len(self.mats), self.K).clone()

    PROFILE_CLASSES = ("clip", "project", "moments", "apply", "outer_states", "outer_weights", "refresh")

    def profile_enable(self, on: bool = True):
        self._check(self.lib.lordo_profile_enable(self._ctx, int(on)), "lordo_profile_enable")

    def profile_read(self, stream=None) -> dict:
        """Milliseconds per kernel class accumulated since the last read (CUDA events)."""
        out = (C.c_float * 8)()
        self._check(self.lib.lordo_profile_read(self._ctx, _stream_handle(stream), out), "lordo_profile_read")
        return {name: float(out[i]) for i, name in enumerate(self.PROFILE_CLASSES)}

    @property
    def launch_count(self) -> int:
        return int(self.lib.lordo_launch_count(self._ctx))

    def close(self):
        if getattr(self, "_ctx", None) is not None and self._ctx.value:
            torch.cuda.synchronize(self.device)
            self.lib.lordo_destroy(self._ctx)
            self._ctx = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
