"""Full-size parity in the launch configuration the benchmark times: the whole layer runs on the device at the
workload's real shape and the oracle checks all of it -- the router and the dispatch plan for all tokens (bit-exact
integers), the auxiliary loss, and every expert's hidden activations, output rows and gradients (the whole of y, dx,
dW_r, dW_in, dW_out), each tensor by its relative Frobenius error and element by element.  Only the wide-expert
workload (8 TFLOP of float64 work for the oracle) samples experts: the fullest, the emptiest non-empty one and one
other.  Properties that hold at any size are asserted as well: dropped tokens give zero rows, experts without
tokens give zero gradients, nothing is NaN.
"""
import numpy as np
import pytest
import torch

from oracle import switch_oracle as so
from paper_2101_03961_b200 import build as sbuild
from paper_2101_03961_b200 import inputs as si
from paper_2101_03961_b200 import switch_moe as sm
from tests.gpu_helpers import (TOL_BF16, TOL_ROUTER, check_flips, check_next_choices, check_second_choice, expert_hidden,
                               follow_relu_flips, rel_err, skip_path_ok, to_np)

pytestmark = pytest.mark.gpu


def _bits_to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


class _ExpertWeights:
    """Expert i's weights as float32, decoded on demand from the bfloat16 bits the device was given (the oracle only
    ever indexes by expert, so host memory stays flat)."""

    def __init__(self, bits: np.ndarray):
        self.bits = bits

    def __getitem__(self, i):
        return si.from_bf16_bits(self.bits[i])


def _run_fullsize(name, seed=0, n_extra=None, residual=False, groups=1, reroute=False, reroute_stages=1):
    sbuild.build()
    cfg = si.CONFIGS[name]
    assert cfg.dtype == si.DTYPE_BF16
    x_np, dy_np = si.gen_x(cfg, seed), si.gen_dy(cfg, seed)
    W_r_np, b_np = si.gen_W_r(cfg, seed), si.gen_router_bias(cfg, seed)
    x, dy = _bits_to_dev(si.to_bf16_bits(x_np)), _bits_to_dev(si.to_bf16_bits(dy_np))
    W_in_bits = si.gen_W_in(cfg, seed, as_bits=True, threads=16)
    W_out_bits = si.gen_W_out(cfg, seed, as_bits=True, threads=16)
    W_in, W_out = _bits_to_dev(W_in_bits), _bits_to_dev(W_out_bits)
    W_r = torch.from_numpy(W_r_np).cuda()
    bias = None if b_np is None else torch.from_numpy(b_np).cuda()
    mcfg = sm.make_config(cfg.T, cfg.d_model, cfg.d_ff, cfg.E, cfg.capacity_factor, cfg.alpha, residual=residual,
                          groups=groups, reroute=reroute, geglu=cfg.geglu, reroute_stages=reroute_stages)
    ws = sm.allocate_workspace(mcfg)
    ws.fill_(0xFF)
    y, dx = torch.full_like(x, float("nan")), torch.full_like(x, float("nan"))
    dW_in, dW_out = torch.full_like(W_in, float("nan")), torch.full_like(W_out, float("nan"))
    dW_r = torch.full_like(W_r, float("nan"))
    aux = torch.zeros(1, device="cuda")
    sm.switch_moe_fwd(mcfg, x, W_r, bias, W_in, W_out, y, aux, ws)
    sm.switch_moe_bwd(mcfg, dy, 1.0, x, W_r, W_in, W_out, y, ws, dx, dW_r, dW_in, dW_out)
    sm.switch_moe_check_device_status(mcfg, ws)
    view = lambda r: sm.switch_moe_workspace_view(mcfg, ws, r)
    T, E, C = cfg.T, cfg.E, sm.switch_moe_capacity(mcfg) * groups      # C: rows per expert in the slot buffers

    # router for all tokens; flips only inside the allowed gap; then the oracle follows the device's choice
    gpu_e = view(sm.WS_EXPERT_INDEX).cpu().numpy().astype(np.int64)
    h = so.router_logits(x_np, W_r_np, b_np)
    p = so.router_probs(h)
    e0, _ = so.top1(p)
    flips = check_flips(gpu_e, {"e": e0, "p": p})
    assert flips <= 8
    assert np.abs(to_np(view(sm.WS_PROBS)).reshape(T, E) - p).max() <= TOL_ROUTER
    alt = None
    if groups == 1:
        plan = so.dispatch_plan(gpu_e, E, so.expert_capacity(T, E, cfg.capacity_factor))
        aux_ref, _, _ = so.load_balance_loss(p, gpu_e, cfg.alpha)
        if reroute:                                          # further stages: next choices, then the grown plan
            gpu_alt = view(sm.WS_SECOND_CHOICE).cpu().numpy().astype(np.int64)
            cap = so.expert_capacity(T, E, cfg.capacity_factor)
            alt = check_next_choices(gpu_alt, p, gpu_e, plan, E, cap)
            for stage_alt in alt:
                before = int(plan["keep"].sum())
                plan = so.reroute_overflow(plan, gpu_e, stage_alt, E, cap)
                assert int(plan["keep"].sum()) > before
            np.testing.assert_array_equal(view(sm.WS_EXPERT_PROC).cpu().numpy(), plan["e_proc"])
    else:                                                    # every group on its own; no expert FFN work here
        plan = so.switch_forward_groups(x_np, W_r_np, {}, {}, cfg.capacity_factor, cfg.alpha, groups,
                                        router_bias=b_np, expert_index=gpu_e, experts=[])
        aux_ref = plan["aux"]
    assert C == groups * so.expert_capacity(T // groups, E, cfg.capacity_factor)
    np.testing.assert_array_equal(view(sm.WS_SLOT).cpu().numpy(), plan["slot"])
    np.testing.assert_array_equal(view(sm.WS_TOKEN_OF_SLOT).cpu().numpy(), plan["token_of_slot"])
    np.testing.assert_array_equal(view(sm.WS_COUNT).cpu().numpy(), plan["count"])
    np.testing.assert_array_equal(view(sm.WS_KEPT).cpu().numpy(), plan["kept"])
    assert abs(float(aux.item()) - aux_ref) <= TOL_ROUTER * aux_ref

    # every expert; or (n_extra given) a sample: the fullest, the emptiest non-empty one and n_extra others
    count = plan["count"]
    nonempty = np.flatnonzero(count > 0)
    if n_extra is None:
        sample = list(range(E))
    else:
        sample = {int(np.argmax(count)), int(nonempty[np.argmin(count[nonempty])])}
        rng = np.random.default_rng(seed)
        sample.update(int(v) for v in rng.choice(nonempty, size=min(n_extra, nonempty.size), replace=False))
        sample = sorted(sample)
    W_in_s, W_out_s = _ExpertWeights(W_in_bits), _ExpertWeights(W_out_bits)
    for i in sample[:2]:                                       # the decoded bits are the seeded generator's values
        np.testing.assert_array_equal(W_in_s[i], si.gen_W_in_expert(cfg, i, seed))
    if groups == 1:
        fwd = so.switch_forward(x_np, W_r_np, W_in_s, W_out_s, cfg.capacity_factor, cfg.alpha, router_bias=b_np,
                                expert_index=gpu_e, experts=sample, residual=residual, reroute=reroute, alt_index=alt,
                                reroute_stages=reroute_stages, geglu=cfg.geglu)
    else:
        fwd = so.switch_forward_groups(x_np, W_r_np, W_in_s, W_out_s, cfg.capacity_factor, cfg.alpha, groups,
                                       router_bias=b_np, expert_index=gpu_e, experts=sample, residual=residual)
    hid = view(sm.WS_H).view(E, C, cfg.d_ff)
    relu_flips = follow_relu_flips(fwd, lambda i, k: to_np(hid[i, :k]), experts=sample)
    if groups == 1:
        bwd = so.switch_backward(fwd, x_np, W_r_np, W_in_s, W_out_s, dy_np, experts=sample)
    else:
        bwd = so.switch_backward_groups(fwd, x_np, W_r_np, W_in_s, W_out_s, dy_np, experts=sample)
    keep = plan["keep"]
    errs = {}
    for i in sample:
        k = int(plan["kept"][i])
        if k == 0:
            continue                                           # zero gradients are asserted below
        tok = plan["token_of_slot"][i * C:i * C + k]           # the expert's tokens in slot order
        tt = torch.from_numpy(tok).cuda()
        errs[f"H[{i}]"] = rel_err(to_np(hid[i, :k]), expert_hidden(fwd, i))
        if residual:
            layer_y = view(sm.WS_LAYER_Y).view(T, cfg.d_model)
            errs[f"layer_y[{i}]"] = rel_err(to_np(layer_y[tt]), fwd["layer_y"][tok])
            assert skip_path_ok(to_np(y[tt]), fwd["y"][tok], fwd["layer_y"][tok], TOL_BF16, sm.BF16)
            assert skip_path_ok(to_np(dx[tt]), bwd["dx"][tok], bwd["dx"][tok] - dy_np[tok].astype(np.float64),
                                TOL_BF16, sm.BF16, roundings=3)
        else:
            errs[f"y[{i}]"] = rel_err(to_np(y[tt]), fwd["y"][tok])
            errs[f"dx[{i}]"] = rel_err(to_np(dx[tt]), bwd["dx"][tok])
        errs[f"dW_in[{i}]"] = rel_err(to_np(dW_in[i]), bwd["dW_in"][i])
        errs[f"dW_out[{i}]"] = rel_err(to_np(dW_out[i]), bwd["dW_out"][i])
        errs[f"dgate[{i}]"] = rel_err(to_np(view(sm.WS_DGATE)[tt]), bwd["dgate"][tok])
    if n_extra is None and not residual:
        # all experts were run: the whole output, the whole input gradient and the router's weight gradient
        errs["y"] = rel_err(to_np(y), fwd["y"])
        errs["dx"] = rel_err(to_np(dx), bwd["dx"])
        errs["dW_r"] = rel_err(to_np(dW_r), bwd["dW_r"])
    bad = {k: v for k, v in errs.items() if not v <= TOL_BF16}
    assert not bad, bad

    # properties that hold at any size
    dropped = torch.from_numpy(np.flatnonzero(~keep)).cuda()
    if dropped.numel():
        assert bool((y[dropped] == (x[dropped] if residual else 0)).all())   # skip path: the input row, bit for bit
    if residual and dropped.numel():
        # a dropped token's dx is dy plus the router's gradient only (checked exactly against the oracle's router)
        some = np.flatnonzero(~keep)[:64]
        assert groups == 1
        G = np.broadcast_to((cfg.alpha * E / T) * fwd["f"][None, :], (some.size, E))
        dh = p[some] * (G - np.sum(p[some] * G, axis=1, keepdims=True))
        want = dy_np[some].astype(np.float64) + dh @ W_r_np.astype(np.float64).T
        assert skip_path_ok(to_np(dx[torch.from_numpy(some).cuda()]), want, dh @ W_r_np.astype(np.float64).T, 1e-3,
                            sm.BF16)
    assert bool(torch.isfinite(y).all()) and bool(torch.isfinite(dx).all()) and bool(torch.isfinite(dW_r).all())
    assert bool(torch.isfinite(dW_in).all()) and bool(torch.isfinite(dW_out).all())
    for i in np.flatnonzero(count == 0):
        assert bool((dW_in[int(i)] == 0).all()) and bool((dW_out[int(i)] == 0).all())
    # dropped tokens receive only the router's gradient: finite and small, never the expert path
    return {"flips": flips, "relu_flips": relu_flips, "dropped": int((~keep).sum()), "errs": errs}


def test_switch_base_full_size():
    out = _run_fullsize("switch_base")
    assert out["dropped"] < 0.01 * 32768                     # well-balanced routing: under 1% dropped


def test_overflow_stress_calibrated_full_size():
    out = _run_fullsize("stress_calibrated")
    assert 0.15 * 32768 < out["dropped"] < 0.40 * 32768


def test_overflow_stress_literal_full_size():
    out = _run_fullsize("stress_literal")
    assert out["dropped"] > 0.8 * 32768                      # a N(0, 2^2) bias overflows almost everything


def test_switch_large_full_size():
    _run_fullsize("switch_large")


def test_wide_expert_full_size():
    _run_fullsize("wide", n_extra=1)                          # sampled experts: the oracle pass would take minutes


def test_overflow_stress_with_the_skip_path_inside_full_size():
    out = _run_fullsize("stress_calibrated", residual=True)
    assert out["dropped"] > 0.15 * 32768


def test_switch_base_in_eight_routing_groups_full_size():
    out = _run_fullsize("switch_base", groups=8)
    assert 0.01 * 32768 < out["dropped"] < 0.2 * 32768        # 40 slots per expert and group: overflow is common


def test_overflow_stress_with_rerouting_full_size():
    out = _run_fullsize("stress_calibrated", reroute=True)
    # capacity factor 1: the experts' slots add up to exactly T, so only part of the 31% overflow finds a second home
    assert out["dropped"] < 0.25 * 32768


def test_overflow_stress_with_three_rerouting_stages_full_size():
    out = _run_fullsize("stress_calibrated", reroute=True, reroute_stages=3)
    # the second, third and fourth choices together leave fewer tokens without a slot than the second alone
    assert out["dropped"] < 0.15 * 32768


def test_geglu_experts_at_the_papers_switch_base_shape_full_size():
    _run_fullsize("geglu_base")


def test_geglu_experts_at_the_papers_switch_large_shape_full_size():
    _run_fullsize("geglu_large")                              # d_ff 2816 = 11 weight-row tiles of 256: an odd count


def test_geglu_experts_at_the_papers_switch_xxl_shape_full_size():
    _run_fullsize("geglu_xxl", n_extra=1)                     # sampled experts: the oracle pass would take minutes


def test_batch_of_131072_tokens_full_size():
    out = _run_fullsize("long_batch")
    assert out["dropped"] < 0.05 * 131072


def test_top2_routing_at_the_switch_base_shape_full_size():
    """Top-2 routing at T=32768, E=128 with the capacity factor 2.0 of the paper's Mixture-of-Experts baselines: the
    plan for all 65536 assignments bit for bit, sampled experts' rows and gradients within tolerance."""
    sbuild.build()
    cfg = si.CONFIGS["switch_base"].with_(capacity_factor=2.0)
    seed = 0
    x_np, dy_np, W_r_np = si.gen_x(cfg, seed), si.gen_dy(cfg, seed), si.gen_W_r(cfg, seed)
    x, dy = _bits_to_dev(si.to_bf16_bits(x_np)), _bits_to_dev(si.to_bf16_bits(dy_np))
    W_in_bits = si.gen_W_in(cfg, seed, as_bits=True, threads=16)
    W_out_bits = si.gen_W_out(cfg, seed, as_bits=True, threads=16)
    W_in, W_out = _bits_to_dev(W_in_bits), _bits_to_dev(W_out_bits)
    W_r = torch.from_numpy(W_r_np).cuda()
    mcfg = sm.make_config(cfg.T, cfg.d_model, cfg.d_ff, cfg.E, cfg.capacity_factor, cfg.alpha, top2=True)
    ws = sm.allocate_workspace(mcfg)
    ws.fill_(0xFF)
    y, dx = torch.full_like(x, float("nan")), torch.full_like(x, float("nan"))
    dW_in, dW_out = torch.full_like(W_in, float("nan")), torch.full_like(W_out, float("nan"))
    dW_r = torch.full_like(W_r, float("nan"))
    aux = torch.zeros(1, device="cuda")
    sm.switch_moe_fwd(mcfg, x, W_r, None, W_in, W_out, y, aux, ws)
    sm.switch_moe_bwd(mcfg, dy, 1.0, x, W_r, W_in, W_out, y, ws, dx, dW_r, dW_in, dW_out)
    sm.switch_moe_check_device_status(mcfg, ws)
    view = lambda r: sm.switch_moe_workspace_view(mcfg, ws, r)
    T, E, C = cfg.T, cfg.E, sm.switch_moe_capacity(mcfg)
    gpu_e = view(sm.WS_EXPERT_INDEX).cpu().numpy().astype(np.int64)
    p = so.router_probs(so.router_logits(x_np, W_r_np))
    first = gpu_e[:T]
    assert check_flips(first, {"e": so.top1(p)[0], "p": p}) <= 8
    second = check_second_choice(gpu_e[T:], p, first, np.ones(T, dtype=bool))
    plan = so.top2_forward(x_np, W_r_np, {}, {}, cfg.capacity_factor, cfg.alpha, first_index=first, second_index=second,
                           experts=[])
    assert C == plan["C"] == 512
    np.testing.assert_array_equal(view(sm.WS_SLOT).cpu().numpy(), plan["slot"])
    np.testing.assert_array_equal(view(sm.WS_TOKEN_OF_SLOT).cpu().numpy(), plan["token_of_slot"])
    np.testing.assert_array_equal(view(sm.WS_COUNT).cpu().numpy(), plan["count_first"])
    np.testing.assert_array_equal(view(sm.WS_KEPT).cpu().numpy(), plan["kept"])
    assert abs(float(aux.item()) - plan["aux"]) <= TOL_ROUTER * plan["aux"]
    assert plan["keep"].mean() > 0.9                           # twice the capacity holds most of the assignments
    kept = plan["kept"]
    sample = list(range(E))                                    # every expert
    W_in_s, W_out_s = _ExpertWeights(W_in_bits), _ExpertWeights(W_out_bits)
    fwd = so.top2_forward(x_np, W_r_np, W_in_s, W_out_s, cfg.capacity_factor, cfg.alpha, first_index=first,
                          second_index=second, experts=sample)
    hid = view(sm.WS_H).view(E, C, cfg.d_ff)
    follow_relu_flips(fwd, lambda i, k: to_np(hid[i, :k]), experts=sample)
    bwd = so.top2_backward(fwd, x_np, W_r_np, W_in_s, W_out_s, dy_np, experts=sample)
    errs = {}
    for i in sample:
        k = int(kept[i])
        v = plan["token_of_slot"][i * C:i * C + k]
        errs[f"H[{i}]"] = rel_err(to_np(hid[i, :k]), np.maximum(fwd["u"][i], 0.0))
        errs[f"dW_in[{i}]"] = rel_err(to_np(dW_in[i]), bwd["dW_in"][i])
        errs[f"dW_out[{i}]"] = rel_err(to_np(dW_out[i]), bwd["dW_out"][i])
        vv = torch.from_numpy(v).cuda()
        errs[f"dgate[{i}]"] = rel_err(to_np(view(sm.WS_DGATE)[vv]), bwd["dgate"][v])
    errs["y"] = rel_err(to_np(y), fwd["y"])
    errs["dx"] = rel_err(to_np(dx), bwd["dx"])
    errs["dW_r"] = rel_err(to_np(dW_r), bwd["dW_r"])
    bad = {k: v for k, v in errs.items() if not v <= TOL_BF16}
    assert not bad, bad
    assert bool(torch.isfinite(y).all()) and bool(torch.isfinite(dx).all()) and bool(torch.isfinite(dW_in).all())
