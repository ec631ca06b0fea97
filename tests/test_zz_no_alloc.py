"""switch_moe_dispatch_plan_static: the dispatch plan for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits -- the device heap belongs to another allocator, or
the call sits on a path that must not synchronise the device -- and they have no workspace to lend either.  This
entry point keeps its scratch in an array compiled into the library.  The test calls it through the C ABI twice in
a row with different routings (the second call sees whatever the first left in the shared array) and requires the
same integers the workspace-based switch_moe_dispatch_plan produces: bit-exact, as for all index work.
This file is collected last so that a failure here cannot hide any other test's result.
"""
import numpy as np
import pytest
import torch

from paper_2101_03961_b200 import build as sbuild
from paper_2101_03961_b200 import switch_moe as sm

pytestmark = pytest.mark.gpu


def _reference_plan(cfg, e_dev):
    ws = sm.allocate_workspace(cfg)
    ws.fill_(0xFF)
    sm.switch_moe_dispatch_plan(cfg, e_dev, None, ws)
    torch.cuda.synchronize()
    return {r: sm.switch_moe_workspace_view(cfg, ws, r).clone()
            for r in (sm.WS_COUNT, sm.WS_KEPT, sm.WS_SLOT, sm.WS_TOKEN_OF_SLOT)}


def test_static_plan_matches_workspace_plan_on_two_calls_in_a_row():
    sbuild.build()
    rng = np.random.default_rng(7)
    # second call: fewer tokens and experts than the first, so stale histogram rows from call one stay in the array
    cases = [(32768, 128, 1.25, 0.5), (5000, 24, 1.0, 0.0)]
    for T, E, cf, skew in cases:
        cfg = sm.make_config(T, 64, 64, E, cf)
        C = sm.switch_moe_capacity(cfg)
        e = rng.integers(0, E, T)
        e[rng.random(T) < skew] = E // 3                      # overflow one expert
        e_dev = torch.from_numpy(e.astype(np.int32)).cuda()
        count = torch.full((E,), -7, dtype=torch.int32, device="cuda")
        kept = torch.full((E,), -7, dtype=torch.int32, device="cuda")
        slot = torch.full((T,), -7, dtype=torch.int32, device="cuda")
        tos = torch.full((E * C,), -7, dtype=torch.int32, device="cuda")
        sm.switch_moe_dispatch_plan_static(cfg, e_dev, count, kept, slot, tos)
        torch.cuda.synchronize()
        ref = _reference_plan(cfg, e_dev)
        assert torch.equal(count, ref[sm.WS_COUNT])
        assert torch.equal(kept, ref[sm.WS_KEPT])
        assert torch.equal(slot, ref[sm.WS_SLOT])
        assert torch.equal(tos, ref[sm.WS_TOKEN_OF_SLOT])
        assert int((slot < 0).sum()) == T - int(kept.sum())


def test_static_plan_rejects_sizes_beyond_its_array():
    import ctypes
    sbuild.build()
    cfg = sm.make_config(65536 + 256, 64, 64, 8, 1.0)
    buf = torch.zeros(8, dtype=torch.int32, device="cuda")
    rc = sm.load_library().switch_moe_dispatch_plan_static(ctypes.byref(cfg), buf.data_ptr(), buf.data_ptr(),
                                                           buf.data_ptr(), buf.data_ptr(), buf.data_ptr(), None)
    assert rc == sm.UNSUPPORTED_SHAPE
    with pytest.raises(sm.SwitchMoeError):
        sm.switch_moe_dispatch_plan_static(cfg, buf, buf, buf, buf, buf)
