"""lordo_clip_coefficient_static: the entry point for callers that cannot allocate device memory.

Some users of the library run where a device allocation is off the table: inside a framework hook
that only lends them fixed buffers, while the job's memory pool is frozen, or so close to the memory
limit that one more cudaMalloc would fail. For them the clip coefficient of a gradient can be had
without a context or a workspace; its scratch is a fixed array inside the library. This test checks
that entry point against the regular path (lordo_inner_step followed by lordo_clip_coefficients on a
one-matrix, one-worker problem), twice in a row on different gradients, because consecutive calls
share the static scratch and the second must not see anything of the first.

The file name makes pytest collect it after every other test file.
"""
import numpy as np
import pytest
import torch

from oracle import lordo_oracle as lo
from paper_2602_04396_b200 import synth
from tests import harness as hz
from tests.harness import RunSpec

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dt", ["f32", "bf16"])
def test_static_clip_coefficient_matches_inner_step(dt):
    from paper_2602_04396_b200 import lordo
    m, n, r, rho = 520, 264, 16, 40.0  # 137280 elements: five partial sums, the last one ragged
    wl = synth.Workload("noalloc", ((m, n, r),), K=1, H=2, rounds=1, grad="gauss", clip_rho=rho, w_dtype=dt, g_dtype=dt,
                        e_dtype=dt)
    opt = hz.make_gpu(RunSpec(wl, refresh=False))
    out = torch.zeros(1, device="cuda", dtype=torch.float32)
    scales = (1.0, 0.05)  # first gradient is clipped, second lies inside the radius
    for step, scale in enumerate(scales):
        G = synth.gradients(wl, 0, 0, step)
        G[0] = (G[0] * np.float32(scale)).astype(np.float32)
        Gd = hz.device_grads(wl, G)
        opt.inner_step(Gd, 0.01, 0.9, 0.9, 0)
        want = float(opt.clip_coefficients()[0, 0])
        lordo.clip_coefficient_static(Gd[0], rho, out)
        got = float(out.item())
        assert abs(got - want) <= 1e-6 * max(want, 1e-30), (step, got, want)
        oracle_c = float(lo.clip_coefficients([np.asarray(hz._np_state(Gd[0]))], rho, 0)[0, 0])  # the definition, on the stored values
        assert abs(got - oracle_c) <= 2e-6 * oracle_c, (step, got, oracle_c)
    assert want == 1.0  # the second call must not carry the first call's large partial sums


def test_static_clip_coefficient_rejects_oversize_and_bad_arguments():
    from paper_2602_04396_b200 import lordo
    lib = lordo.load_library()
    limit = lib.lordo_clip_coefficient_static_max_count()
    assert limit == 16384 * 32768
    out = torch.zeros(1, device="cuda", dtype=torch.float32)
    g = torch.zeros(64, device="cuda", dtype=torch.float32)
    import ctypes as C
    call = lambda count: lib.lordo_clip_coefficient_static(C.c_void_p(g.data_ptr()), 0, count, 1.0, C.c_void_p(out.data_ptr()), None)
    assert call(limit + 8) == 8  # LORDO_ERR_UNSUPPORTED: beyond the static scratch, nothing launched
    assert call(60) == 1         # not a multiple of 8
    assert call(64) == 0
    torch.cuda.synchronize()
    assert float(out.item()) == 1.0  # zero gradient: norm 0, coefficient min(1, rho/1e-6) = 1
