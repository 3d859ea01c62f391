"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, validates configurations and sizes its workspace."""
import ctypes as C
import os
import re

import pytest

from paper_2602_04396_b200 import build as lbuild
from paper_2602_04396_b200 import lordo

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    lbuild.build()
    return lordo.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "lordo.h")).read()
    declared = sorted(set(re.findall(r"LORDO_API\s+[\w\s\*]+?\b(lordo_\w+)\s*\(", header)))
    assert len(declared) >= 15
    assert sorted(lordo.EXPORTS) == declared
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings(lib):
    assert lib.lordo_status_string(0) == b"ok"
    assert b"order" in lib.lordo_status_string(4)


def test_workspace_query_and_validation(lib):
    cfg, _keep = lordo.make_config([(256, 256, 16)], 2, 4, clip_rho=1.0)
    small = lordo.query_workspace(cfg)
    cfg2, _keep2 = lordo.make_config([(256, 256, 16)] * 3, 2, 4, clip_rho=1.0)
    assert lordo.query_workspace(cfg2) > small > 0
    # g^ and U~ workspaces alone: 2 * K * r * n floats
    assert small >= 2 * 2 * 16 * 256 * 4
    bad = [
        ([(256, 252, 16)], dict(), 3),           # n not a multiple of 8
        ([(256, 256, 12)], dict(), 3),           # r not a multiple of 8
        ([(16, 256, 32)], dict(), 2),            # r > m
        ([(256, 256, 16)], dict(beta2=1.0), 1),  # beta2 out of range
        ([(256, 256, 16)], dict(power_iters=9), 1),
        ([(256, 256, 16)], dict(variant=5), 1),
        ([(256, 256, 16)], dict(time_buffer=2), 1),
        ([(256, 256, 16)], dict(oversample=4), 1),                  # not a multiple of 8
        ([(256, 256, 16)], dict(oversample=8, warm_start=1), 8),    # needs a fresh sketch
        ([(256, 24, 16)], dict(oversample=16), 2),                  # r + p > n
        ([(1024, 1024, 512)], dict(oversample=96), 2),              # r + p > 600
        ([(252, 256, 16)], dict(sides=[1]), 3),                     # projected from the right: m not a multiple of 8
        ([(256, 256, 16)], dict(sides=[2]), 1),                     # no such side
        ([(256, 256, 16)], dict(sides=[1], time_buffer=1), 8),      # not available from the right
        ([(256, 256, 16)], dict(sides=[1], oversample=8), 8),
    ]
    for mats, kw, code in bad:
        cfg, _k = lordo.make_config(mats, 2, 4, **kw)
        with pytest.raises(lordo.LordoError) as ei:
            lordo.query_workspace(cfg)
        assert ei.value.status == code
    # both options cost workspace: the time buffers (K r n floats) and the wider sketch
    c0, _k0 = lordo.make_config([(256, 256, 16)], 2, 4)
    c1, _k1 = lordo.make_config([(256, 256, 16)], 2, 4, time_buffer=1)
    c2, _k2 = lordo.make_config([(256, 256, 16)], 2, 4, oversample=8)
    base = lordo.query_workspace(c0)
    assert lordo.query_workspace(c1) >= base + 2 * 16 * 256 * 4
    assert lordo.query_workspace(c2) > base
    cfg, _k = lordo.make_config([(256, 256, 16)], 65, 4)
    with pytest.raises(lordo.LordoError):
        lordo.query_workspace(cfg)
    # projected from the right, the low-rank arrays of a tall matrix have m columns instead of n
    tall_l, _kl = lordo.make_config([(1024, 128, 16)], 2, 4, check_mode=1)
    tall_r, _kr = lordo.make_config([(1024, 128, 16)], 2, 4, check_mode=1, sides=[1])
    assert lordo.query_workspace(tall_r) > lordo.query_workspace(tall_l)


def test_null_arguments_are_rejected(lib):
    assert lib.lordo_query_workspace(None, None) == 1
    assert lib.lordo_inner_step(None, None, 0.1, 0.9, 0.9, 0, None) == 1
    assert lib.lordo_outer_step(None, None) == 1
    assert lib.lordo_destroy(None) == 1
    assert lib.lordo_launch_count(None) == -1
