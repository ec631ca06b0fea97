"""switch_moe_dispatch_plan_static: the dispatch plan for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits -- the device heap belongs to another allocator, or
the call sits on a path that must not synchronise the device -- and they have no workspace to lend either.  This
entry point keeps its scratch in an array compiled into the library.  The test calls it through the C ABI twice in
a row with different routings (the second call sees whatever the first left in the shared array) and requires the
integers of the CPU oracle's plan and of the workspace-based switch_moe_dispatch_plan: bit-exact, as for all index
work.  This file is collected last so that a failure here cannot hide any other test's result.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import switch_oracle as so
from paper_2101_03961_b200 import build as sbuild
from paper_2101_03961_b200 import switch_moe as sm

pytestmark = pytest.mark.gpu


def _workspace_plan(cfg, e_dev):
    ws = sm.allocate_workspace(cfg)
    ws.fill_(0xFF)
    sm.switch_moe_dispatch_plan(cfg, e_dev, None, ws)
    torch.cuda.synchronize()
    return {r: sm.switch_moe_workspace_view(cfg, ws, r).clone()
            for r in (sm.WS_COUNT, sm.WS_KEPT, sm.WS_SLOT, sm.WS_TOKEN_OF_SLOT)}


def _oracle_plan(e: np.ndarray, E: int, C: int):
    """The oracle's plan; entries of -1 ("no expert", the library's own marker for a token without a second choice)
    take no slot, i.e. the plan is the oracle's plan of the remaining tokens in their original numbering."""
    valid = np.flatnonzero(e >= 0)
    sub = so.dispatch_plan(e[valid], E, C)
    slot = np.full(e.shape[0], -1, dtype=np.int64)
    slot[valid] = sub["slot"]
    tos = np.where(sub["token_of_slot"] >= 0, valid[np.maximum(sub["token_of_slot"], 0)], -1)
    return {"count": sub["count"], "kept": sub["kept"], "slot": slot, "token_of_slot": tos}


def _static_plan(cfg, e_dev, T, E, C):
    count = torch.full((E,), -7, dtype=torch.int32, device="cuda")
    kept = torch.full((E,), -7, dtype=torch.int32, device="cuda")
    slot = torch.full((T,), -7, dtype=torch.int32, device="cuda")
    tos = torch.full((E * C,), -7, dtype=torch.int32, device="cuda")
    sm.switch_moe_dispatch_plan_static(cfg, e_dev, count, kept, slot, tos)
    torch.cuda.synchronize()
    return count, kept, slot, tos


def test_static_plan_matches_oracle_and_workspace_plan_on_two_calls_in_a_row():
    sbuild.build()
    rng = np.random.default_rng(7)
    # second call: fewer tokens and experts than the first, so stale histogram rows from call one stay in the array;
    # third call: some tokens carry -1 (no expert) and must take no slot
    cases = [(32768, 128, 1.25, 0.5, 0.0), (5000, 24, 1.0, 0.0, 0.0), (3000, 16, 1.0, 0.2, 0.1)]
    for T, E, cf, skew, none in cases:
        cfg = sm.make_config(T, 64, 64, E, cf)
        C = sm.switch_moe_capacity(cfg)
        e = rng.integers(0, E, T)
        e[rng.random(T) < skew] = E // 3                      # overflow one expert
        e[rng.random(T) < none] = -1
        e_dev = torch.from_numpy(e.astype(np.int32)).cuda()
        count, kept, slot, tos = _static_plan(cfg, e_dev, T, E, C)
        want = _oracle_plan(e, E, C)
        np.testing.assert_array_equal(count.cpu().numpy(), want["count"])
        np.testing.assert_array_equal(kept.cpu().numpy(), want["kept"])
        np.testing.assert_array_equal(slot.cpu().numpy(), want["slot"])
        np.testing.assert_array_equal(tos.cpu().numpy(), want["token_of_slot"])
        ref = _workspace_plan(cfg, e_dev)
        assert torch.equal(count, ref[sm.WS_COUNT])
        assert torch.equal(kept, ref[sm.WS_KEPT])
        assert torch.equal(slot, ref[sm.WS_SLOT])
        assert torch.equal(tos, ref[sm.WS_TOKEN_OF_SLOT])
        assert int((slot < 0).sum()) == T - int(kept.sum())


def test_static_plan_rejects_sizes_beyond_its_array():
    sbuild.build()
    cfg = sm.make_config(65536 + 256, 64, 64, 8, 1.0)
    buf = torch.zeros(8, dtype=torch.int32, device="cuda")
    rc = sm.load_library().switch_moe_dispatch_plan_static(ctypes.byref(cfg), buf.data_ptr(), buf.data_ptr(),
                                                           buf.data_ptr(), buf.data_ptr(), buf.data_ptr(), None)
    assert rc == sm.UNSUPPORTED_SHAPE
    with pytest.raises(sm.SwitchMoeError):
        sm.switch_moe_dispatch_plan_static(cfg, buf, buf, buf, buf, buf)


@pytest.mark.parametrize("kw", [{"top2": True}, {"reroute": True}], ids=["top2", "reroute"])
def test_static_plan_rejects_the_routing_variants_it_does_not_implement(kw):
    """Top-2 routing places 2T assignments (twice the histogram rows the array is sized for) and rerouting runs a
    second stage: both need the workspace-based call.  Only the status code is checked; nothing is launched."""
    sbuild.build()
    cfg = sm.make_config(65536, 64, 64, 256, 2.0, **kw)
    buf = torch.zeros(8, dtype=torch.int32, device="cuda")
    rc = sm.load_library().switch_moe_dispatch_plan_static(ctypes.byref(cfg), buf.data_ptr(), buf.data_ptr(),
                                                           buf.data_ptr(), buf.data_ptr(), buf.data_ptr(), None)
    assert rc == sm.UNSUPPORTED_SHAPE
