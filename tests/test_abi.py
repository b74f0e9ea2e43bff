"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
the header declares, validates configurations, and reports sizes."""
import ctypes
import os
import re

import pytest

from paper_2302_08545_b200 import thc, workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
T4_30 = W.TABLES[(4, 30)]


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "thc.h")).read()
    declared = set(re.findall(r"^\s*(?:int|const char \*)\s*(thc_\w+)\s*\(", header, flags=re.M))
    assert declared == set(thc.EXPORTS)
    L = thc.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert "sm_100a" in thc.version()


def _ctx(**kw):
    base = dict(bits=4, granularity=30, table=T4_30, t_p=W.T_P["1/32"], log2_block=20,
                seed=W.THC_SEED, workers=8)
    base.update(kw)
    return thc.Context(**base)


def test_sizes_match_the_paper_prototype_ratios():
    c = _ctx()
    s = c.sizes(25_557_032, 8)
    assert s.d_pad == 26_214_400 and s.nblocks == 25
    assert s.packed_bytes == s.d_pad // 2          # 32-bit -> 4-bit: x8
    assert s.sum_bytes == s.d_pad                  # 8-bit sums: x4
    assert s.acc_bits == 8                         # 8 * 30 = 240 <= 255
    assert _ctx(workers=9).sizes(100, 1).acc_bits == 16
    assert _ctx(workers=9, acc_bits=32).sizes(100, 1).acc_bits == 32


@pytest.mark.parametrize("kw", [
    dict(bits=5), dict(bits=0), dict(granularity=14), dict(table=(1,) + T4_30[1:]),
    dict(table=T4_30[:-1] + (29,)), dict(table=(0, 3, 3) + T4_30[3:]), dict(t_p=0.0),
    dict(t_p=float("nan")), dict(log2_block=2), dict(log2_block=23), dict(in_dtype=7),
    dict(workers=0), dict(workers=65), dict(acc_bits=12), dict(workers=9, acc_bits=8),
    dict(range_mode=2),
])
def test_invalid_configurations_are_rejected(kw):
    with pytest.raises(thc.ThcError) as e:
        _ctx(**kw)
    assert e.value.code == thc.THC_EINVAL


def test_unsupported_granularity():
    with pytest.raises(thc.ThcError) as e:
        _ctx(bits=8, granularity=300, table=tuple(range(255)) + (300,))
    assert e.value.code == thc.THC_EUNSUPPORTED


def test_range_mode_sizes_and_limits():
    """Exact-range contexts keep two floats per RHT block (minima, then maxima), never take
    the fused scales path, and accept fp32 input only."""
    c = _ctx(range_mode=1)
    s = c.sizes(25_557_032, 8)
    assert s.scales_count == 2 * s.nblocks and s.fused_scales == 0
    n = _ctx().sizes(25_557_032, 8)
    assert n.scales_count == n.nblocks and n.fused_scales == 1
    assert _ctx().sizes(25_557_032, 14).fused_scales == 0        # ring would not fit in L2
    assert _ctx(log2_block=16).sizes(25_557_032, 8).fused_scales == 0
    with pytest.raises(thc.ThcError) as e:
        _ctx(range_mode=1, in_dtype=thc.THC_BF16)
    assert e.value.code == thc.THC_EUNSUPPORTED


def test_sizes_argument_checks_and_strerror():
    c = _ctx()
    with pytest.raises(thc.ThcError):
        c.sizes(0, 1)
    with pytest.raises(thc.ThcError):
        c.sizes(10, 0)
    with pytest.raises(thc.ThcError):
        c.sizes(10, 65)
    assert "workspace" in thc.strerror(thc.THC_EWORKSPACE)
    assert thc.strerror(0) == "ok"


def test_launch_without_a_device_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    c = _ctx(log2_block=10)
    buf = (ctypes.c_char * 4096)()
    addr = (ctypes.addressof(buf) + 15) & ~15
    with pytest.raises(thc.ThcError) as e:
        c.aggregate([addr], 1024, addr, stream=0)
    assert e.value.code == thc.THC_ECUDA
