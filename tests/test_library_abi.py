"""The C-ABI library loads, exports every symbol the header declares, and its host-only calls behave."""
import ctypes
import os
import re

import pytest

from paper_2101_03961_b200 import build as sbuild
from paper_2101_03961_b200 import switch_moe as sm

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    sbuild.build()
    return sm.load_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "switch_moe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(switch_moe_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    declared = _declared_symbols()
    assert len(declared) >= 10
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(sm.EXPORTED_SYMBOLS) == declared


def test_capacity_follows_eq3(lib):
    for T, E, cf, C in [(512, 8, 1.0, 64), (32768, 128, 1.25, 320), (32768, 64, 1.0, 512), (16384, 64, 1.25, 320),
                        (10, 4, 1.25, 3), (8, 1, 2.0, 8)]:
        assert sm.switch_moe_capacity(sm.make_config(T, 64, 64, E, cf)) == C
    assert sm.switch_moe_capacity(sm.make_config(512, 64, 64, 8, 1.0, capacity_override=17)) == 17
    # several routing groups: Eq. 3 on the tokens of one group
    assert sm.switch_moe_capacity(sm.make_config(32768, 768, 3072, 128, 1.25, groups=8)) == 40
    assert sm.switch_moe_capacity(sm.make_config(2048, 64, 64, 8, 1.0, groups=2)) == 128


def test_workspace_size_is_positive_and_grows(lib):
    a = sm.switch_moe_workspace_bytes(sm.make_config(512, 64, 256, 8, 1.0, dtype=sm.F32))
    b = sm.switch_moe_workspace_bytes(sm.make_config(32768, 768, 3072, 128, 1.25))
    assert 0 < a < b
    slots = 128 * 320
    assert b >= 2 * slots * (768 + 3072) * 2                   # X_d, H, dY_d, dH in bf16


@pytest.mark.parametrize("kw,status", [
    (dict(T=0), sm.INVALID_ARGUMENT), (dict(E=0), sm.INVALID_ARGUMENT), (dict(capacity_factor=0.0), sm.INVALID_ARGUMENT),
    (dict(E=257), sm.UNSUPPORTED_SHAPE), (dict(d_model=100), sm.UNSUPPORTED_SHAPE),
    (dict(T=4, E=8, capacity_factor=1.0), sm.INVALID_ARGUMENT),          # capacity would be 0
    (dict(dtype=7), sm.INVALID_ARGUMENT),
    (dict(T=2048, groups=3), sm.INVALID_ARGUMENT),                       # T not a multiple of the group count
    (dict(T=1000, groups=2), sm.UNSUPPORTED_SHAPE),                      # groups of 500 tokens: not a multiple of 256
    (dict(T=131072, groups=2), sm.UNSUPPORTED_SHAPE),
    (dict(T=2048, groups=-1), sm.INVALID_ARGUMENT),
])
def test_bad_configs_are_rejected(lib, kw, status):
    base = dict(T=512, d_model=64, d_ff=256, E=8, capacity_factor=1.0)
    base.update(kw)
    cfg = sm.make_config(**base)
    out = ctypes.c_size_t(0)
    assert lib.switch_moe_workspace_bytes(ctypes.byref(cfg), ctypes.byref(out)) == status
    with pytest.raises(sm.SwitchMoeError):
        sm.switch_moe_workspace_bytes(cfg)


def test_null_pointers_are_rejected_without_touching_the_device(lib):
    cfg = sm.make_config(512, 64, 256, 8, 1.0, dtype=sm.F32)
    assert lib.switch_moe_fwd(ctypes.byref(cfg), None, None, None, None, None, None, None, None, 0, None) \
        == sm.INVALID_ARGUMENT
    assert lib.switch_moe_capacity(ctypes.byref(cfg), None) == sm.INVALID_ARGUMENT
    assert lib.switch_moe_capacity(None, None) == sm.INVALID_ARGUMENT
    # a workspace that is too small is reported before anything is launched
    assert lib.switch_moe_router_fwd(ctypes.byref(cfg), 1024, 1024, None, 1024, 16, None) == sm.WORKSPACE_TOO_SMALL


def test_status_strings(lib):
    assert sm.status_string(0) == "ok"
    assert "workspace" in sm.status_string(sm.WORKSPACE_TOO_SMALL)
    assert sm.status_string(-99) == "unknown status"


def test_launch_count_is_reported(lib):
    assert sm.switch_moe_launches_per_step(sm.make_config(512, 64, 256, 8, 1.0, dtype=sm.F32)) == 16
    # bf16 default path: the router's epilogue leaves the probabilities' column sums and the plan's histograms, and the
    # two products of dH share one launch
    assert sm.switch_moe_launches_per_step(sm.make_config(512, 64, 256, 8, 1.0)) == 14
    # options add launches: four plan kernels per rerouting stage, one product kernel for input jitter; GEGLU gating and
    # expert dropout live in the GEMM epilogues on this path and add none
    assert sm.switch_moe_launches_per_step(sm.make_config(512, 64, 256, 8, 1.0, reroute=True, input_jitter=True,
                                                          geglu=True, expert_dropout=0.4)) == 14 + 4 + 1
    assert sm.switch_moe_launches_per_step(sm.make_config(512, 64, 256, 8, 1.0, geglu=True)) == 14
    assert sm.switch_moe_launches_per_step(sm.make_config(512, 64, 256, 8, 1.0, reroute=True, reroute_stages=3)) == 14 + 12
    # the fp32 path gates, and drops hidden units, in element-wise kernels both ways
    assert sm.switch_moe_launches_per_step(sm.make_config(512, 64, 256, 8, 1.0, dtype=sm.F32, geglu=True)) == 16 + 2
    assert sm.switch_moe_launches_per_step(sm.make_config(512, 64, 256, 8, 1.0, dtype=sm.F32, geglu=True,
                                                          expert_dropout=0.4)) == 16 + 2 + 2
