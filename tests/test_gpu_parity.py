"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded inputs.

Integer work (expert counts, slots, drop masks, inverse maps) must match bit for bit.  Floating point is held to
the tolerances in gpu_helpers (router 1e-5; bf16 tensors 2e-2; all-fp32 layer 2e-4), each tensor by its relative
Frobenius error and element by element, |a - b| <= 2 tol (rms_i(b) + |b|) with the local rms of gpu_helpers.
Argmax flips are counted and allowed only inside a top-2 probability gap of 1e-4; the oracle then follows the
device's expert choice, because a single flip moves every later slot of two experts.  The sign decision of the
ReLU derivative is treated the same way (gpu_helpers.follow_relu_flips).
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import switch_oracle as so
from paper_2101_03961_b200 import inputs as si
from paper_2101_03961_b200 import switch_moe as sm
from tests.gpu_helpers import (TOL_BF16, TOL_F32, TOL_ROUTER, GpuLayer, check_flips, expert_hidden, follow_relu_flips,
                               oracle_following, rel_err, skip_path_ok, to_np)

pytestmark = pytest.mark.gpu

TINY = si.CONFIGS["tiny"]
# bf16 cases that span several tiles and ragged tails in every dimension (T, C, d, f not multiples of the tiles)
MID = si.SwitchConfig("mid", 2048, 128, 256, 8, 1.25)
RAGGED = si.SwitchConfig("ragged", 1999, 192, 320, 5, 1.25, bias_std=0.3)
MANY = si.SwitchConfig("many_experts", 4096, 64, 128, 96, 1.0, bias_std=0.2)


def _stack(d):
    return np.stack([d[i] for i in range(len(d))])


# ---------------------------------------------------------------------------------------------- router (staged)
@pytest.mark.parametrize("cfg", [TINY, MID, RAGGED, MANY, si.SwitchConfig("e1", 300, 64, 64, 1, 1.0),
                                 si.SwitchConfig("e256", 1024, 64, 64, 256, 2.0)], ids=lambda c: c.name)
def test_router_forward_matches_oracle(cfg):
    data = si.gen_layer(cfg, seed=0)
    g = GpuLayer(cfg, data)
    sm.switch_moe_router_fwd(g.cfg, g.x, g.W_r, g.bias, g.ws)
    torch.cuda.synchronize()
    h = so.router_logits(data["x"], data["W_r"], data.get("router_bias"))
    p = so.router_probs(h)
    e, gate = so.top1(p)
    probs = to_np(g.view(sm.WS_PROBS)).reshape(cfg.T, cfg.E)
    assert np.abs(probs - p).max() <= TOL_ROUTER
    assert rel_err(probs, p) <= TOL_ROUTER
    np.testing.assert_allclose(probs.sum(1), 1.0, atol=1e-5)
    gpu_e = g.expert_index()
    flips = check_flips(gpu_e, {"e": e, "p": p})
    assert flips <= max(2, cfg.T // 1000)
    gpu_gate = to_np(g.view(sm.WS_GATE))
    np.testing.assert_allclose(gpu_gate, p[np.arange(cfg.T), gpu_e], rtol=TOL_ROUTER, atol=1e-7)


def test_router_ties_go_to_lowest_expert():
    cfg = si.SwitchConfig("ties", 256, 64, 64, 16, 1.0)
    data = si.gen_layer(cfg, seed=1)
    data["W_r"][:] = 0.0
    g = GpuLayer(cfg, data)
    g.fwd()
    assert (g.expert_index() == 0).all()
    np.testing.assert_allclose(to_np(g.view(sm.WS_GATE)), 1.0 / 16, rtol=1e-6)
    slot = g.view(sm.WS_SLOT).cpu().numpy()
    C = g.C
    assert slot.tolist() == [t if t < C else -1 for t in range(cfg.T)]          # exactly the first C tokens kept
    assert abs(float(g.aux.item()) - cfg.alpha) <= 1e-6 * cfg.alpha + 1e-9        # P uniform => aux = alpha
    y = to_np(g.y)
    assert np.all(y[C:] == 0.0) and np.isfinite(y).all()


# ---------------------------------------------------------------------------------------------- dispatch (staged)
def _plan_case(name, T, E, C, e):
    return name, T, E, C, np.asarray(e, dtype=np.int32)


def _plan_cases():
    rng = np.random.default_rng(0)
    cases = [
        _plan_case("uniform", 4096, 16, 256, rng.integers(0, 16, 4096)),
        _plan_case("ragged_T", 1999, 5, 499, rng.integers(0, 5, 1999)),
        _plan_case("all_one_expert", 3000, 8, 375, np.full(3000, 3)),
        _plan_case("round_robin", 2048, 64, 32, np.arange(2048) % 64),
        _plan_case("capacity_1", 700, 7, 1, rng.integers(0, 7, 700)),
        _plan_case("e256", 5000, 256, 19, rng.integers(0, 256, 5000)),
    ]
    skew = rng.integers(0, 32, 32768)
    skew[rng.random(32768) < 0.5] = 7
    cases.append(_plan_case("skewed_32k", 32768, 32, 1024, skew))
    return cases


@pytest.mark.parametrize("case", _plan_cases(), ids=lambda c: c[0])
def test_dispatch_plan_is_bit_exact_given_oracle_routing(case):
    _, T, E, C, e = case
    cfg = sm.make_config(T, 64, 64, E, 1.0, capacity_override=C)
    ws = sm.allocate_workspace(cfg)
    ws.fill_(0xFF)
    sm.switch_moe_dispatch_plan(cfg, torch.from_numpy(e).cuda(), None, ws)
    torch.cuda.synchronize()
    plan = so.dispatch_plan(e, E, C)
    v = lambda r: sm.switch_moe_workspace_view(cfg, ws, r).cpu().numpy().astype(np.int64)
    np.testing.assert_array_equal(v(sm.WS_COUNT), plan["count"])
    np.testing.assert_array_equal(v(sm.WS_KEPT), plan["kept"])
    np.testing.assert_array_equal(v(sm.WS_SLOT), plan["slot"])
    np.testing.assert_array_equal(v(sm.WS_TOKEN_OF_SLOT), plan["token_of_slot"])
    np.testing.assert_array_equal(v(sm.WS_SLOT) >= 0, plan["keep"])


def test_dispatch_plan_is_deterministic():
    rng = np.random.default_rng(5)
    e = torch.from_numpy(rng.integers(0, 128, 32768).astype(np.int32)).cuda()
    cfg = sm.make_config(32768, 64, 64, 128, 1.0)
    ws = sm.allocate_workspace(cfg)
    outs = []
    for _ in range(3):
        ws.fill_(0xFF)
        sm.switch_moe_dispatch_plan(cfg, e, None, ws)
        torch.cuda.synchronize()
        outs.append(sm.switch_moe_workspace_view(cfg, ws, sm.WS_SLOT).clone())
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])


# ---------------------------------------------------------------------------------------------- whole layer
def _check_layer(cfg, gemm_path, tol, seed=0, d_aux=1.0, capacity_override=0, residual=False, groups=1,
                 reroute=False, noise_eps=0.0, jitter_eps=0.0, geglu=False, dropout=0.0, reroute_stages=1):
    if geglu:                                                  # W_in = [W_0 | W_1]: twice the columns
        cfg = cfg.with_(geglu=True)
    data = si.gen_layer(cfg, seed=seed)
    if jitter_eps:
        data["router_jitter"] = si.gen_router_jitter(cfg, jitter_eps, seed)
    if dropout:
        rows = cfg.E * so.expert_capacity(cfg.T, cfg.E, cfg.capacity_factor)
        data["expert_keep"], data["expert_dropout"] = si.gen_expert_keep(cfg, rows, dropout, seed), dropout
    if noise_eps:
        data["router_noise"] = si.gen_router_noise(cfg, noise_eps, seed)
    g = GpuLayer(cfg, data, gemm_path=gemm_path, capacity_override=capacity_override, residual=residual,
                 groups=groups, reroute=reroute, geglu=geglu, reroute_stages=reroute_stages)
    g.fwd()
    gpu_e = g.expert_index()
    cap = capacity_override if capacity_override else None
    gpu_alt = g.view(sm.WS_SECOND_CHOICE).cpu().numpy().astype(np.int64) if reroute else None
    fwd = oracle_following(cfg, data, gpu_e, capacity=cap, residual=residual, groups=groups, gpu_alt=gpu_alt,
                           geglu=geglu)
    if reroute:
        np.testing.assert_array_equal(g.view(sm.WS_EXPERT_PROC).cpu().numpy(), fwd["e_proc"])
        np.testing.assert_allclose(to_np(g.view(sm.WS_GATE))[fwd["keep"]], fwd["g"][fwd["keep"]], rtol=2e-5)
    assert g.C == fwd["C"]                                     # Eq. 3 for one routing group
    E, C = cfg.E, g.C * groups                                 # rows per expert in the slot buffers
    # integer state: bit exact
    np.testing.assert_array_equal(g.view(sm.WS_SLOT).cpu().numpy(), fwd["slot"])
    np.testing.assert_array_equal(g.view(sm.WS_COUNT).cpu().numpy(), fwd["count"])
    np.testing.assert_array_equal(g.view(sm.WS_KEPT).cpu().numpy(), fwd["kept"])
    np.testing.assert_array_equal(g.view(sm.WS_TOKEN_OF_SLOT).cpu().numpy(), fwd["token_of_slot"])
    # router and loss
    assert rel_err(to_np(g.view(sm.WS_PROBS)).reshape(cfg.T, E), fwd["p"]) <= TOL_ROUTER
    assert abs(float(g.aux.item()) - fwd["aux"]) <= TOL_ROUTER * abs(fwd["aux"])
    np.testing.assert_allclose(to_np(g.view(sm.WS_PSUM)), fwd["p"].sum(0), rtol=TOL_ROUTER)
    # dispatched tokens and hidden activations, slot by slot
    xd = to_np(g.view(sm.WS_XD)).reshape(E, C, cfg.d_model)
    hid = to_np(g.view(sm.WS_H)).reshape(E, C, cfg.d_ff)
    x64 = np.asarray(data["x"], dtype=np.float64)
    errs = {}
    for i in range(E):
        k = int(fwd["kept"][i])
        if k == 0:
            continue
        tok = fwd["token_of_slot"][i * C:i * C + k]
        np.testing.assert_array_equal(xd[i, :k], x64[tok])
        errs[f"H[{i}]"] = rel_err(hid[i, :k], expert_hidden(fwd, i))
    follow_relu_flips(fwd, lambda i, k: hid[i, :k])            # ReLU signs inside the gap: the oracle follows the device
    y = to_np(g.y)
    assert np.isfinite(y).all()
    if residual:
        # dropped tokens leave the layer unchanged, bit for bit; kept ones: the layer term (kept in the workspace
        # without the skip path) is held to the usual tolerance, the sum to the rounding of its storage type
        np.testing.assert_array_equal(y[~fwd["keep"]], to_np(g.x)[~fwd["keep"]])
        layer_y = to_np(g.view(sm.WS_LAYER_Y)).reshape(cfg.T, cfg.d_model)
        errs["layer_y"] = rel_err(layer_y[fwd["keep"]], fwd["layer_y"][fwd["keep"]])
        assert skip_path_ok(y, fwd["y"], fwd["layer_y"], tol, cfg.dtype)
    else:
        assert np.all(y[~fwd["keep"]] == 0.0)                  # dropped tokens: zero rows
        errs["y"] = rel_err(y, fwd["y"])

    g.bwd(d_aux=d_aux)
    backward = so.switch_backward_groups if groups > 1 else so.switch_backward
    bwd = backward(fwd, data["x"], data["W_r"], data["W_in"], data["W_out"], data["dy"], d_aux=d_aux)
    kept_tok = np.flatnonzero(fwd["keep"])
    errs["dgate"] = rel_err(to_np(g.view(sm.WS_DGATE))[kept_tok], bwd["dgate"][kept_tok])
    if residual:
        assert skip_path_ok(to_np(g.dx), bwd["dx"], bwd["dx"] - np.asarray(data["dy"], dtype=np.float64), tol, cfg.dtype,
                            roundings=3)
    else:
        errs["dx"] = rel_err(to_np(g.dx), bwd["dx"])
    errs["dW_r"] = rel_err(to_np(g.dW_r), bwd["dW_r"])
    dW_in, dW_out = to_np(g.dW_in), to_np(g.dW_out)
    assert np.isfinite(dW_in).all() and np.isfinite(dW_out).all() and np.isfinite(to_np(g.dx)).all()
    errs["dW_in"] = rel_err(dW_in, _stack(bwd["dW_in"]))
    errs["dW_out"] = rel_err(dW_out, _stack(bwd["dW_out"]))
    for i in range(E):
        if fwd["kept"][i] == 0:                                # expert without tokens: exactly zero gradients
            assert np.all(dW_in[i] == 0) and np.all(dW_out[i] == 0)
    bad = {k: v for k, v in errs.items() if not v <= tol}
    assert not bad, (bad, errs)
    LAST_ORACLE["fwd"] = fwd                                   # for tests that assert more about the routing
    return errs


LAST_ORACLE = {}


def test_tiny_fp32_layer_matches_oracle():
    _check_layer(TINY, sm.GEMM_DEFAULT, TOL_F32)


@pytest.mark.parametrize("cfg", [MID, RAGGED, MANY], ids=lambda c: c.name)
def test_bf16_layer_on_fp32_fma_path_matches_oracle(cfg):
    _check_layer(cfg, sm.GEMM_SIMT, TOL_BF16)


@pytest.mark.parametrize("cfg", [MID, RAGGED, MANY], ids=lambda c: c.name)
def test_bf16_layer_on_tensor_cores_matches_oracle(cfg):
    _check_layer(cfg, sm.GEMM_DEFAULT, TOL_BF16, d_aux=0.5)


@pytest.mark.parametrize("cfg", [MID, RAGGED], ids=lambda c: c.name)
def test_bf16_layer_on_single_cta_tensor_core_path_matches_oracle(cfg):
    _check_layer(cfg, sm.GEMM_TC_1CTA, TOL_BF16, d_aux=0.5)


@pytest.mark.parametrize("cfg,path,tol", [(TINY, sm.GEMM_DEFAULT, TOL_F32), (MID, sm.GEMM_SIMT, TOL_BF16),
                                          (MID, sm.GEMM_DEFAULT, TOL_BF16), (RAGGED, sm.GEMM_DEFAULT, TOL_BF16),
                                          (MANY, sm.GEMM_DEFAULT, TOL_BF16)],
                         ids=["tiny_f32", "mid_fma", "mid_tc", "ragged_tc", "many_tc"])
def test_layer_with_the_skip_path_inside_matches_oracle(cfg, path, tol):
    """y = x + g E(x) fused into the combine step, dx = dy + ... fused into the scatter step (Fig. 2, Section 2.2)."""
    _check_layer(cfg, path, tol, residual=True)


GROUPED = si.SwitchConfig("grouped", 2048, 128, 256, 8, 1.0, bias_std=0.3)
GROUPED_F32 = si.SwitchConfig("grouped_f32", 512, 64, 128, 4, 0.75, dtype=si.DTYPE_F32)


@pytest.mark.parametrize("cfg,path,tol,groups,residual", [
    (GROUPED_F32, sm.GEMM_DEFAULT, TOL_F32, 2, False), (GROUPED, sm.GEMM_SIMT, TOL_BF16, 4, False),
    (GROUPED, sm.GEMM_DEFAULT, TOL_BF16, 2, False), (GROUPED, sm.GEMM_DEFAULT, TOL_BF16, 8, False),
    (GROUPED, sm.GEMM_TC_1CTA, TOL_BF16, 4, False), (GROUPED, sm.GEMM_DEFAULT, TOL_BF16, 4, True)],
    ids=["f32_g2", "fma_g4", "tc_g2", "tc_g8", "tc1_g4", "tc_g4_skip"])
def test_several_routing_groups_in_one_call_match_oracle(cfg, path, tol, groups, residual):
    """Each group of T / G rows is routed on its own (capacity, f, P), experts shared, loss = mean over groups."""
    errs = _check_layer(cfg, path, tol, groups=groups, residual=residual, d_aux=0.7)
    assert errs


def test_group_count_limits_are_enforced():
    for kw in (dict(T=2048, groups=3), dict(T=2048 + 256, groups=2), dict(T=1000, groups=2),
               dict(groups=2, expert_dropout=0.2)):          # expert dropout: one routing group only
        base = dict(T=2048, d_model=128, d_ff=256, E=8, capacity_factor=1.0)
        base.update(kw)
        with pytest.raises(sm.SwitchMoeError):
            sm.switch_moe_workspace_bytes(sm.make_config(**base))


OVERFLOW = si.SwitchConfig("overflow", 2048, 128, 256, 8, 1.0, bias_std=0.5)
OVERFLOW_F32 = si.SwitchConfig("overflow_f32", 512, 64, 128, 4, 0.75, dtype=si.DTYPE_F32, bias_std=0.5)


@pytest.mark.parametrize("cfg,path,tol,residual", [
    (OVERFLOW_F32, sm.GEMM_DEFAULT, TOL_F32, False), (OVERFLOW, sm.GEMM_SIMT, TOL_BF16, False),
    (OVERFLOW, sm.GEMM_DEFAULT, TOL_BF16, False), (MANY, sm.GEMM_DEFAULT, TOL_BF16, False),
    (RAGGED, sm.GEMM_TC_1CTA, TOL_BF16, False), (OVERFLOW, sm.GEMM_DEFAULT, TOL_BF16, True)],
    ids=["f32", "fma", "tc", "many_tc", "ragged_tc1", "tc_skip"])
def test_rerouting_of_overflowed_tokens_matches_oracle(cfg, path, tol, residual):
    """Stage 2 of No-Token-Left-Behind routing (Appendix B): overflow goes to the second choice where it has room."""
    data = si.gen_layer(cfg, seed=0)
    plain = so.switch_forward(data["x"], data["W_r"], data["W_in"], data["W_out"], cfg.capacity_factor, cfg.alpha,
                              router_bias=data.get("router_bias"), experts=[])
    assert (~plain["keep"]).sum() > 0.03 * cfg.T               # the case does overflow
    _check_layer(cfg, path, tol, reroute=True, residual=residual, d_aux=0.7)


@pytest.mark.parametrize("cfg,path,tol,stages", [
    (OVERFLOW_F32, sm.GEMM_DEFAULT, TOL_F32, 2), (OVERFLOW, sm.GEMM_SIMT, TOL_BF16, 3),
    (OVERFLOW, sm.GEMM_DEFAULT, TOL_BF16, 3), (MANY, sm.GEMM_DEFAULT, TOL_BF16, 4),
    (RAGGED, sm.GEMM_DEFAULT, TOL_BF16, 16)],
    ids=["f32_2", "fma_3", "tc_3", "many_tc_4", "ragged_tc_16"])
def test_iterated_rerouting_matches_oracle(cfg, path, tol, stages):
    """No-Token-Left-Behind routing repeated (Appendix B, the figure's caption): stage k offers the tokens still
    without a slot to the expert with their k-th highest probability.  Each stage must keep more tokens than the
    one before while any are waiting and slots are free; the whole layer is compared as everywhere else."""
    _check_layer(cfg, path, tol, reroute=True, reroute_stages=stages, d_aux=0.7)
    fwd = LAST_ORACLE["fwd"]
    data = si.gen_layer(cfg, seed=0)
    one = so.switch_forward(data["x"], data["W_r"], data["W_in"], data["W_out"], cfg.capacity_factor, cfg.alpha,
                            router_bias=data.get("router_bias"), experts=[], reroute=True)
    assert fwd["keep"].sum() > one["keep"].sum()               # the later stages placed tokens stage 2 could not
    if stages >= cfg.E - 1:                                    # every token has tried every expert
        assert fwd["keep"].sum() == min(cfg.T, cfg.E * fwd["C"])


def test_more_rerouting_stages_than_the_config_allows_are_refused():
    with pytest.raises(sm.SwitchMoeError):
        sm.switch_moe_workspace_bytes(sm.make_config(2048, 128, 256, 8, 1.0, reroute=True, reroute_stages=17))
    assert sm.switch_moe_workspace_bytes(sm.make_config(2048, 128, 256, 8, 1.0, reroute_stages=17)) > 0   # ignored without the flag


@pytest.mark.parametrize("cfg,path,tol", [(TINY, sm.GEMM_DEFAULT, TOL_F32), (MID, sm.GEMM_SIMT, TOL_BF16),
                                          (MID, sm.GEMM_DEFAULT, TOL_BF16), (MANY, sm.GEMM_DEFAULT, TOL_BF16),
                                          (si.SwitchConfig("e160", 1024, 128, 128, 160, 1.25), sm.GEMM_DEFAULT, TOL_BF16)],
                         ids=["tiny_f32", "mid_fma", "mid_tc", "many_tc", "e160_tc_generic"])
def test_exploration_noise_on_the_logits_matches_oracle(cfg, path, tol):
    """uniform(1 - eps, 1 + eps) noise added to the router logits (router pseudo-code), passed in as an input."""
    data = si.gen_layer(cfg, seed=0)
    quiet = so.switch_forward(data["x"], data["W_r"], data["W_in"], data["W_out"], cfg.capacity_factor, cfg.alpha,
                              router_bias=data.get("router_bias"), experts=[])
    noisy = so.switch_forward(data["x"], data["W_r"], data["W_in"], data["W_out"], cfg.capacity_factor, cfg.alpha,
                              router_bias=data.get("router_bias"), experts=[],
                              router_noise=si.gen_router_noise(cfg, 0.5, 0))
    assert (quiet["e"] != noisy["e"]).mean() > 0.05           # the noise does change the routing
    _check_layer(cfg, path, tol, noise_eps=0.5)


@pytest.mark.parametrize("cfg,path,tol,residual", [
    (TINY, sm.GEMM_DEFAULT, TOL_F32, False), (MID, sm.GEMM_SIMT, TOL_BF16, False), (MID, sm.GEMM_DEFAULT, TOL_BF16, False),
    (RAGGED, sm.GEMM_DEFAULT, TOL_BF16, False), (MANY, sm.GEMM_DEFAULT, TOL_BF16, True)],
    ids=["tiny_f32", "mid_fma", "mid_tc", "ragged_tc", "many_tc_skip"])
def test_multiplicative_jitter_on_the_router_input_matches_oracle(cfg, path, tol, residual):
    """The router sees x . u (Appendix C, text), the experts see x; dW_r uses x . u and the router's dx is scaled by u."""
    _check_layer(cfg, path, tol, jitter_eps=0.25, residual=residual, d_aux=0.7)


def test_jitter_flag_without_the_factors_is_refused():
    cfg = sm.make_config(MID.T, MID.d_model, MID.d_ff, MID.E, MID.capacity_factor, input_jitter=True)
    ws = sm.allocate_workspace(cfg)
    x = torch.zeros(MID.T, MID.d_model, dtype=torch.bfloat16, device="cuda")
    W_r = torch.zeros(MID.d_model, MID.E, device="cuda")
    with pytest.raises(sm.SwitchMoeError):
        sm.switch_moe_router_fwd(cfg, x, W_r, None, ws)


@pytest.mark.parametrize("cfg,path,tol,residual", [
    (TINY, sm.GEMM_DEFAULT, TOL_F32, False), (MID, sm.GEMM_SIMT, TOL_BF16, False), (MID, sm.GEMM_DEFAULT, TOL_BF16, False),
    (RAGGED, sm.GEMM_DEFAULT, TOL_BF16, False), (MANY, sm.GEMM_DEFAULT, TOL_BF16, True)],
    ids=["tiny_f32", "mid_fma", "mid_tc", "ragged_tc", "many_tc_skip"])
def test_geglu_experts_match_oracle(cfg, path, tol, residual):
    """hidden = GELU(x W_0) . (x W_1) (Table 9): one grouped GEMM with 2 d_ff columns; the gating and its derivative
    sit in the GEMM epilogues on the CTA-pair path and in element-wise kernels on the others.  The ragged case has
    d_ff = 320: the last CTA pair of the gated GEMM1 holds hidden units beyond d_ff, which must not be stored."""
    _check_layer(cfg, path, tol, geglu=True, residual=residual, d_aux=0.7)


def test_rerouting_is_refused_with_several_routing_groups():
    with pytest.raises(sm.SwitchMoeError):
        sm.switch_moe_workspace_bytes(sm.make_config(2048, 128, 256, 8, 1.0, groups=2, reroute=True))


def test_skip_path_is_refused_on_the_single_cta_validation_path():
    cfg = sm.make_config(MID.T, MID.d_model, MID.d_ff, MID.E, MID.capacity_factor, gemm_path=sm.GEMM_TC_1CTA,
                         residual=True)
    with pytest.raises(sm.SwitchMoeError):
        sm.switch_moe_workspace_bytes(cfg)


def test_tensor_core_layer_with_two_token_tiles_per_expert():
    # capacity 600 > 256: experts' tokens are cut into several N tiles of the paired-CTA GEMM
    cfg = si.SwitchConfig("big_capacity", 2400, 128, 320, 4, 1.0, bias_std=0.5)
    _check_layer(cfg, sm.GEMM_DEFAULT, TOL_BF16, seed=5)


def test_tensor_core_layer_with_empty_and_overflowing_experts():
    # a strong bias leaves some experts empty and overflows others; capacity not a multiple of any tile
    cfg = si.SwitchConfig("skewed", 3000, 128, 192, 12, 1.0, bias_std=2.0)
    errs = _check_layer(cfg, sm.GEMM_DEFAULT, TOL_BF16, seed=3)
    assert errs


def test_tensor_core_layer_single_expert_is_dense_ffn():
    cfg = si.SwitchConfig("dense", 512, 128, 256, 1, 1.0)
    data = si.gen_layer(cfg, seed=2)
    g = GpuLayer(cfg, data)
    g.fwd()
    x, W_in, W_out = (np.asarray(data[k], dtype=np.float64) for k in ("x", "W_in", "W_out"))
    dense = np.maximum(x @ W_in[0], 0) @ W_out[0]
    assert rel_err(to_np(g.y), dense) <= TOL_BF16
    np.testing.assert_allclose(to_np(g.view(sm.WS_GATE)), 1.0)


def test_capacity_override_is_honoured():
    _check_layer(MID, sm.GEMM_DEFAULT, TOL_BF16, capacity_override=200)


# ---------------------------------------------------------------------------------------------- router backward (staged)
@pytest.mark.parametrize("cfg,path", [
    (TINY, sm.GEMM_SIMT), (MID.with_(dtype=si.DTYPE_F32), sm.GEMM_SIMT), (RAGGED, sm.GEMM_SIMT),
    (RAGGED, sm.GEMM_DEFAULT), (MID, sm.GEMM_DEFAULT), (MANY, sm.GEMM_DEFAULT),
    (si.SwitchConfig("e256_bwd", 1500, 64, 64, 256, 2.0), sm.GEMM_DEFAULT),
], ids=lambda v: v.name if hasattr(v, "name") else ("tensor_core_router" if v == sm.GEMM_DEFAULT else "fma_router"))
def test_router_backward_given_identical_gate_gradient(cfg, path):
    data = si.gen_layer(cfg, seed=4)
    g = GpuLayer(cfg, data, gemm_path=path)
    g.fwd()
    gpu_e = g.expert_index()
    fwd = oracle_following(cfg, data, gpu_e, experts=[])
    rng = np.random.default_rng(4)
    dgate = rng.standard_normal(cfg.T).astype(np.float32)
    dxr = torch.full_like(g.x, float("nan"))
    sm.switch_moe_router_bwd(g.cfg, g.x, g.W_r, torch.from_numpy(dgate).cuda(), 0.7, g.ws, dxr, g.dW_r)
    torch.cuda.synchronize()
    p_gpu = to_np(g.view(sm.WS_PROBS)).reshape(cfg.T, cfg.E)
    ref = so.router_backward_given_dgate(p_gpu, gpu_e, fwd["keep"], fwd["count"], dgate, data["x"], data["W_r"],
                                         cfg.alpha, d_aux=0.7)
    assert rel_err(to_np(g.view(sm.WS_DLOGITS)).reshape(cfg.T, cfg.E), ref["dh"]) <= TOL_ROUTER
    assert rel_err(to_np(g.dW_r), ref["dW_r"]) <= TOL_ROUTER
    tol_dx = TOL_ROUTER if cfg.dtype == si.DTYPE_F32 else 4e-3          # bf16 output rounding
    assert rel_err(to_np(dxr), ref["dx_router"]) <= tol_dx


# ---------------------------------------------------------------------------------------------- error paths
def test_undersized_workspace_and_misaligned_pointers_are_rejected():
    import ctypes
    cfg = sm.make_config(512, 64, 256, 8, 1.0)
    ws = sm.allocate_workspace(cfg)
    lib = sm.load_library()
    x = torch.zeros(512, 64, dtype=torch.bfloat16, device="cuda")
    W_r = torch.zeros(64, 8, device="cuda")
    rc = lib.switch_moe_router_fwd(ctypes.byref(cfg), x.data_ptr(), W_r.data_ptr(), None, ws.data_ptr(),
                                   ws.numel() - 1, None)
    assert rc == sm.WORKSPACE_TOO_SMALL
    rc = lib.switch_moe_router_fwd(ctypes.byref(cfg), x.data_ptr() + 2, W_r.data_ptr(), None, ws.data_ptr(),
                                   ws.numel(), None)
    assert rc == sm.UNSUPPORTED_SHAPE
    rc = lib.switch_moe_router_fwd(ctypes.byref(cfg), x.data_ptr(), W_r.data_ptr(), None, ws.data_ptr() + 16,
                                   ws.numel(), None)
    assert rc == sm.UNSUPPORTED_SHAPE


def test_a_recorded_device_timeout_is_reported_by_the_status_check():
    """The failure path of the bounded device waits, host half: a kernel that gives up a wait records a code in the
    workspace's status words and returns; switch_moe_check_device_status must then answer DEVICE_TIMEOUT with the
    raw words.  The words are written here from the host (no kernel is made to wait), and a clean workspace must
    read as OK again after the next forward pass has cleared them."""
    cfg = MID
    data = si.gen_layer(cfg, seed=0)
    g = GpuLayer(cfg, data)
    g.fwd()
    assert sm.switch_moe_check_device_status(g.cfg, g.ws)[0] == 0
    status = g.view(sm.WS_STATUS)
    status[:3] = torch.tensor([23, 5, 1], dtype=torch.int32, device="cuda")     # code, block, barrier phase
    info = (ctypes.c_int32 * 16)()
    rc = sm.load_library().switch_moe_check_device_status(ctypes.byref(g.cfg), g.ws.data_ptr(), info, None)
    assert rc == sm.DEVICE_TIMEOUT
    assert list(info)[:3] == [23, 5, 1]
    with pytest.raises(sm.SwitchMoeError) as err:
        sm.switch_moe_check_device_status(g.cfg, g.ws)
    assert err.value.status == sm.DEVICE_TIMEOUT and "timed out" in str(err.value)
    g.fwd()                                                    # the forward pass clears the words first
    assert sm.switch_moe_check_device_status(g.cfg, g.ws)[0] == 0


def test_tokens_without_an_expert_take_no_slot():
    """A caller-supplied index of -1 is "no expert" (the library's own marker, e.g. for a token without a second
    choice): it casts no vote and gets slot -1."""
    T, E, C = 3000, 16, 150
    rng = np.random.default_rng(3)
    e = rng.integers(0, E, T)
    bad = rng.random(T) < 0.1
    e_in = np.where(bad, -1, e).astype(np.int32)
    cfg = sm.make_config(T, 64, 64, E, 1.0, capacity_override=C)
    ws = sm.allocate_workspace(cfg)
    ws.fill_(0xFF)
    sm.switch_moe_dispatch_plan(cfg, torch.from_numpy(e_in).cuda(), None, ws)
    torch.cuda.synchronize()
    valid = np.flatnonzero(~bad)
    sub = so.dispatch_plan(e[valid], E, C)                     # the oracle's plan of the tokens that have an expert
    slot = np.full(T, -1, dtype=np.int64)
    slot[valid] = sub["slot"]
    v = lambda r: sm.switch_moe_workspace_view(cfg, ws, r).cpu().numpy().astype(np.int64)
    np.testing.assert_array_equal(v(sm.WS_COUNT), sub["count"])
    np.testing.assert_array_equal(v(sm.WS_KEPT), sub["kept"])
    np.testing.assert_array_equal(v(sm.WS_SLOT), slot)
    np.testing.assert_array_equal(v(sm.WS_TOKEN_OF_SLOT),
                                  np.where(sub["token_of_slot"] >= 0, valid[np.maximum(sub["token_of_slot"], 0)], -1))


# ---------------------------------------------------------------------------------------------- host-buffer step
@pytest.mark.parametrize("extra_streams", [False, True], ids=["one_stream", "copy_streams"])
def test_step_with_host_activations_equals_device_calls(extra_streams):
    cfg = MID
    data = si.gen_layer(cfg, seed=6)
    g = GpuLayer(cfg, data)
    g.fwd()
    g.bwd()
    y_ref, dx_ref, aux_ref = g.y.clone(), g.dx.clone(), float(g.aux.item())
    dW_in_ref = g.dW_in.clone()
    xh, dyh = g.x.cpu().pin_memory(), g.dy.cpu().pin_memory()
    yh, dxh = torch.empty_like(xh).pin_memory(), torch.empty_like(xh).pin_memory()
    auxh = torch.zeros(1).pin_memory()
    x_dev, dy_dev = torch.zeros_like(g.x), torch.zeros_like(g.x)
    g.y.fill_(float("nan")); g.dx.fill_(float("nan")); g.dW_in.fill_(float("nan"))
    up, down = (torch.cuda.Stream(), torch.cuda.Stream()) if extra_streams else (None, None)
    for _ in range(2):                                       # twice: the call must leave nothing pending behind it
        sm.switch_moe_step_host(g.cfg, xh, dyh, 1.0, g.W_r, g.bias, g.W_in, g.W_out, x_dev, dy_dev, g.y, g.dx, g.aux,
                                g.dW_r, g.dW_in, g.dW_out, yh, dxh, auxh, g.ws, None, up, down)
    assert torch.equal(yh.cuda(), y_ref) and torch.equal(dxh.cuda(), dx_ref)
    assert float(auxh.item()) == aux_ref
    assert torch.equal(g.dW_in, dW_in_ref)


def test_steps_kept_in_flight_give_the_results_of_the_blocking_call():
    """switch_moe_step_host_enqueue with two staging slots and different inputs per step: every step's host results
    equal those of a blocking call on the same inputs."""
    cfg = MID
    layers = [GpuLayer(cfg, si.gen_layer(cfg, seed=s)) for s in (7, 8, 9)]
    g = layers[0]                                            # its weights, workspace and gradient buffers serve all steps
    hosts = []
    for other in layers:
        xh, dyh = other.x.cpu().pin_memory(), other.dy.cpu().pin_memory()
        yh, dxh = torch.empty_like(xh).pin_memory(), torch.empty_like(xh).pin_memory()
        auxh = torch.zeros(1).pin_memory()
        x_dev, dy_dev = torch.zeros_like(g.x), torch.zeros_like(g.x)
        sm.switch_moe_step_host(g.cfg, xh, dyh, 1.0, g.W_r, g.bias, g.W_in, g.W_out, x_dev, dy_dev, g.y, g.dx, g.aux,
                                g.dW_r, g.dW_in, g.dW_out, yh, dxh, auxh, g.ws)
        hosts.append({"xh": xh, "dyh": dyh, "y": yh.clone(), "dx": dxh.clone(), "aux": float(auxh.item()),
                      "dW_in": g.dW_in.clone()})
    slots = [{"x": torch.zeros_like(g.x), "dy": torch.zeros_like(g.x), "y": torch.zeros_like(g.x),
              "dx": torch.zeros_like(g.x), "aux": torch.zeros(1, device="cuda"), "done": None} for _ in range(2)]
    main, up, down = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    outs = []
    for i, h in enumerate(hosts):
        sl = slots[i % 2]
        yh, dxh = torch.empty_like(h["xh"]).pin_memory(), torch.empty_like(h["xh"]).pin_memory()
        auxh = torch.zeros(1).pin_memory()
        done = torch.cuda.Event()
        sm.switch_moe_step_host_enqueue(g.cfg, h["xh"], h["dyh"], 1.0, g.W_r, g.bias, g.W_in, g.W_out, sl["x"],
                                        sl["dy"], sl["y"], sl["dx"], sl["aux"], g.dW_r, g.dW_in, g.dW_out, yh, dxh,
                                        auxh, g.ws, main, up, down, sl["done"], done)
        sl["done"] = done
        outs.append((yh, dxh, auxh, done))
    for (yh, dxh, auxh, done), h in zip(outs, hosts):
        done.synchronize()
        assert torch.equal(yh, h["y"]) and torch.equal(dxh, h["dx"]) and float(auxh.item()) == h["aux"]
    torch.cuda.synchronize()
    assert torch.equal(g.dW_in, hosts[-1]["dW_in"])           # the gradient buffers hold the last step's gradients
    sm.switch_moe_check_device_status(g.cfg, g.ws)
    # the copy streams and the completion event are required
    h = hosts[0]
    rc = sm.load_library().switch_moe_step_host_enqueue(
        ctypes.byref(g.cfg), h["xh"].data_ptr(), h["dyh"].data_ptr(), 1.0, g.W_r.data_ptr(), None, g.W_in.data_ptr(),
        g.W_out.data_ptr(), slots[0]["x"].data_ptr(), slots[0]["dy"].data_ptr(), slots[0]["y"].data_ptr(),
        slots[0]["dx"].data_ptr(), slots[0]["aux"].data_ptr(), g.dW_r.data_ptr(), g.dW_in.data_ptr(),
        g.dW_out.data_ptr(), outs[0][0].data_ptr(), outs[0][1].data_ptr(), outs[0][2].data_ptr(), g.ws.data_ptr(),
        g.ws.numel(), main.cuda_stream, None, None, None, None)
    assert rc == sm.INVALID_ARGUMENT


def test_forward_and_backward_can_be_captured_in_a_cuda_graph():
    """Both calls only enqueue work on the caller's stream (no allocation, no synchronisation), so a step can be
    captured once and replayed; the replay on new inputs gives what direct calls give."""
    cfg = MID
    g = GpuLayer(cfg, si.gen_layer(cfg, seed=11))
    g.fwd()
    g.bwd()                                                  # first calls outside the capture (one-time set-up)
    other = si.gen_layer(cfg, seed=12)
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            sm.switch_moe_fwd(g.cfg, g.x, g.W_r, g.bias, g.W_in, g.W_out, g.y, g.aux, g.ws, side)
            sm.switch_moe_bwd(g.cfg, g.dy, 1.0, g.x, g.W_r, g.W_in, g.W_out, g.y, g.ws, g.dx, g.dW_r, g.dW_in, g.dW_out,
                              side)
    torch.cuda.synchronize()
    from tests.gpu_helpers import to_dev
    g.x.copy_(to_dev(other["x"], cfg.dtype))
    g.dy.copy_(to_dev(other["dy"], cfg.dtype))
    for t in (g.y, g.dx, g.dW_in, g.dW_out):
        t.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    got = [t.clone() for t in (g.y, g.dx, g.dW_r, g.dW_in, g.dW_out, g.aux)]
    g.fwd()
    g.bwd()
    for a, b in zip(got, (g.y, g.dx, g.dW_r, g.dW_in, g.dW_out, g.aux)):
        assert torch.equal(a, b)


@pytest.mark.parametrize("cfg", [
    si.SwitchConfig("five_tokens", 5, 64, 64, 2, 1.0),                       # fewer tokens than any tile
    si.SwitchConfig("one_token", 1, 64, 64, 1, 1.0),                         # the smallest call there is
    si.SwitchConfig("max_experts", 2048, 64, 128, 256, 2.0, bias_std=0.2),   # E = 256, the library's limit
    si.SwitchConfig("more_experts_than_tokens", 128, 64, 64, 256, 4.0),      # most experts stay empty, capacity 2
    si.SwitchConfig("capacity_is_everything", 300, 64, 128, 3, 3.0),         # cf = E: capacity = T, nothing can drop
], ids=lambda c: c.name)
def test_extreme_shapes_match_oracle(cfg):
    errs = _check_layer(cfg, sm.GEMM_DEFAULT, TOL_BF16, d_aux=0.5)
    assert errs


# ---------------------------------------------------------------------------------------------- top-2 routing
def _check_top2(cfg, gemm_path, tol, seed=0, d_aux=0.7, residual=False, expect_mix=True):
    from tests.gpu_helpers import check_second_choice
    data = si.gen_layer(cfg, seed=seed)
    g = GpuLayer(cfg, data, gemm_path=gemm_path, top2=True, residual=residual)
    g.fwd()
    T, E, C = cfg.T, cfg.E, g.C
    gpu_e = g.expert_index()
    assert gpu_e.shape == (2 * T,)
    first, second = gpu_e[:T], gpu_e[T:]
    probe = so.switch_forward(data["x"], data["W_r"], data["W_in"], data["W_out"], cfg.capacity_factor, cfg.alpha,
                              router_bias=data.get("router_bias"), experts=[])
    check_flips(first, probe)
    second = check_second_choice(second, probe["p"], first, np.ones(T, dtype=bool))
    fwd = so.top2_forward(data["x"], data["W_r"], data["W_in"], data["W_out"], cfg.capacity_factor, cfg.alpha,
                          router_bias=data.get("router_bias"), first_index=first, second_index=second,
                          residual=residual)
    assert C == fwd["C"]
    keep = fwd["keep"]
    if expect_mix:                                             # the case is meant to exercise both:
        assert keep[T:].any() and (~keep).any()               # second choices do get slots, and some assignments overflow
    np.testing.assert_array_equal(g.view(sm.WS_SLOT).cpu().numpy(), fwd["slot"])
    np.testing.assert_array_equal(g.view(sm.WS_TOKEN_OF_SLOT).cpu().numpy(), fwd["token_of_slot"])
    np.testing.assert_array_equal(g.view(sm.WS_COUNT).cpu().numpy(), fwd["count_first"])   # f counts first choices
    np.testing.assert_array_equal(g.view(sm.WS_KEPT).cpu().numpy(), fwd["kept"])
    assert rel_err(to_np(g.view(sm.WS_PROBS)).reshape(T, E), fwd["p"]) <= TOL_ROUTER
    assert abs(float(g.aux.item()) - fwd["aux"]) <= TOL_ROUTER * abs(fwd["aux"])
    np.testing.assert_allclose(to_np(g.view(sm.WS_GATE))[keep], fwd["g"][keep], rtol=2e-5)
    xd = to_np(g.view(sm.WS_XD)).reshape(E, C, cfg.d_model)
    hid = to_np(g.view(sm.WS_H)).reshape(E, C, cfg.d_ff)
    x64 = np.asarray(data["x"], dtype=np.float64)
    errs = {}
    for i in range(E):
        k = int(fwd["kept"][i])
        if k == 0:
            continue
        v = fwd["token_of_slot"][i * C:i * C + k]
        np.testing.assert_array_equal(xd[i, :k], x64[fwd["tok_of"][v]])
        errs[f"H[{i}]"] = rel_err(hid[i, :k], np.maximum(fwd["u"][i], 0.0))
    follow_relu_flips(fwd, lambda i, k: hid[i, :k])
    y = to_np(g.y)
    assert np.isfinite(y).all()
    both_dropped = ~keep[:T] & ~keep[T:]
    if residual:                                               # such a token leaves the layer unchanged, bit for bit
        np.testing.assert_array_equal(y[both_dropped], to_np(g.x)[both_dropped])
        assert skip_path_ok(y, fwd["y"], fwd["layer_y"], tol, cfg.dtype)
    else:
        assert np.all(y[both_dropped] == 0.0)
        errs["y"] = rel_err(y, fwd["y"])
    g.bwd(d_aux=d_aux)
    bwd = so.top2_backward(fwd, data["x"], data["W_r"], data["W_in"], data["W_out"], data["dy"], d_aux=d_aux)
    kept_v = np.flatnonzero(keep)
    errs["dgate"] = rel_err(to_np(g.view(sm.WS_DGATE))[kept_v], bwd["dgate"][kept_v])
    if residual:
        assert skip_path_ok(to_np(g.dx), bwd["dx"], bwd["dx"] - np.asarray(data["dy"], dtype=np.float64), tol, cfg.dtype)
    else:
        errs["dx"] = rel_err(to_np(g.dx), bwd["dx"])
    errs["dW_r"] = rel_err(to_np(g.dW_r), bwd["dW_r"])
    errs["dW_in"] = rel_err(to_np(g.dW_in), _stack(bwd["dW_in"]))
    errs["dW_out"] = rel_err(to_np(g.dW_out), _stack(bwd["dW_out"]))
    bad = {k: v for k, v in errs.items() if not v <= tol}
    assert not bad, (bad, errs)


TOP2 = si.SwitchConfig("top2", 2048, 128, 256, 8, 1.5, bias_std=0.3)
TOP2_F32 = si.SwitchConfig("top2_f32", 512, 64, 128, 4, 1.5, dtype=si.DTYPE_F32, bias_std=0.3)


@pytest.mark.parametrize("cfg,path,tol", [(TOP2_F32, sm.GEMM_DEFAULT, TOL_F32), (TOP2, sm.GEMM_SIMT, TOL_BF16),
                                          (TOP2, sm.GEMM_DEFAULT, TOL_BF16), (TOP2, sm.GEMM_TC_1CTA, TOL_BF16),
                                          (si.SwitchConfig("top2_many", 4096, 64, 128, 96, 2.0, bias_std=0.2),
                                           sm.GEMM_DEFAULT, TOL_BF16)],
                         ids=["f32", "fma", "tc", "tc1", "many_tc"])
def test_top2_routing_matches_oracle(cfg, path, tol):
    """y = p_a E_a(x) + p_b E_b(x): first choices placed before second choices, one capacity, f from the first choice."""
    _check_top2(cfg, path, tol)


def test_top2_is_refused_with_the_options_it_does_not_combine_with():
    for kw in (dict(reroute=True), dict(groups=2), dict(T=2000), dict(geglu=True), dict(expert_dropout=0.2),
               dict(input_jitter=True)):
        base = dict(T=2048, d_model=128, d_ff=256, E=8, capacity_factor=1.5, top2=True)
        base.update(kw)
        with pytest.raises(sm.SwitchMoeError):
            sm.switch_moe_workspace_bytes(sm.make_config(**base))


@pytest.mark.parametrize("kw", [dict(), dict(residual=True), dict(reroute=True), dict(top2=True), dict(geglu=True)],
                         ids=["plain", "skip", "reroute", "top2", "geglu"])
def test_results_are_bitwise_reproducible(kw):
    """No floating-point atomics and fixed reduction orders everywhere: two runs on the same inputs give the same bits,
    whatever ran in between."""
    cfg = si.SwitchConfig("repro", 2048, 128, 256, 8, 1.0, bias_std=0.5)
    if kw.get("geglu"):
        cfg = cfg.with_(geglu=True)
    data = si.gen_layer(cfg, seed=3)
    g = GpuLayer(cfg, data, **{k: v for k, v in kw.items() if k != "geglu"})
    outs = []
    for rep in range(3):
        for t in (g.y, g.dx, g.dW_r, g.dW_in, g.dW_out):
            t.fill_(float("nan"))
        if rep == 1:
            g.ws.fill_(0x5A)                                  # different stale workspace contents
            g.view(sm.WS_STATUS).zero_()
        g.fwd()
        g.bwd(d_aux=0.3)
        outs.append([t.clone() for t in (g.y, g.dx, g.dW_r, g.dW_in, g.dW_out, g.aux)])
    for other in outs[1:]:
        for a, b in zip(outs[0], other):
            assert torch.equal(a, b)


def test_options_combine():
    """Rerouting + the skip path + GEGLU experts + logit noise + input jitter in one call; several groups + GEGLU;
    several groups + the skip path + input jitter."""
    cfg = si.SwitchConfig("combo", 2048, 128, 256, 8, 1.0, bias_std=0.5)
    _check_layer(cfg, sm.GEMM_DEFAULT, TOL_BF16, reroute=True, residual=True, geglu=True, noise_eps=0.3, jitter_eps=0.2,
                 d_aux=0.4)
    _check_layer(cfg, sm.GEMM_SIMT, TOL_BF16, reroute=True, residual=True, geglu=True, noise_eps=0.3, jitter_eps=0.2,
                 d_aux=0.4)
    _check_layer(si.SwitchConfig("combo_groups", 2048, 128, 256, 8, 1.0, bias_std=0.3), sm.GEMM_DEFAULT, TOL_BF16,
                 groups=4, geglu=True, noise_eps=0.3, d_aux=0.4)
    _check_layer(si.SwitchConfig("combo_groups", 2048, 128, 256, 8, 1.0, bias_std=0.3), sm.GEMM_DEFAULT, TOL_BF16,
                 groups=2, residual=True, jitter_eps=0.2, d_aux=0.4)


def test_top2_with_a_single_expert_has_no_second_choice():
    cfg = si.SwitchConfig("top2_one_expert", 256, 64, 64, 1, 1.0)
    data = si.gen_layer(cfg, seed=0)
    g = GpuLayer(cfg, data, top2=True)
    g.fwd()
    g.bwd()
    e = g.expert_index()
    assert np.all(e[:256] == 0) and np.all(e[256:] == -1)
    assert np.all(g.view(sm.WS_SLOT).cpu().numpy()[256:] == -1)
    plain = GpuLayer(cfg, data)
    plain.fwd()
    plain.bwd()
    for a, b in ((g.y, plain.y), (g.dx, plain.dx), (g.dW_in, plain.dW_in), (g.dW_out, plain.dW_out), (g.dW_r, plain.dW_r)):
        assert torch.equal(a, b)


@pytest.mark.parametrize("cfg,path,tol,kw", [
    (TINY, sm.GEMM_DEFAULT, TOL_F32, {}), (MID, sm.GEMM_SIMT, TOL_BF16, {}), (MID, sm.GEMM_DEFAULT, TOL_BF16, {}),
    (RAGGED, sm.GEMM_DEFAULT, TOL_BF16, dict(reroute=True)), (MANY, sm.GEMM_DEFAULT, TOL_BF16, dict(geglu=True, residual=True)),
    (MID, sm.GEMM_SIMT, TOL_BF16, dict(geglu=True)), (MID, sm.GEMM_DEFAULT, TOL_BF16, dict(geglu=True, reroute=True, reroute_stages=2))],
    ids=["tiny_f32", "mid_fma", "mid_tc", "ragged_tc_reroute", "many_tc_geglu_skip", "mid_fma_geglu", "mid_tc_geglu_reroute2"])
def test_expert_dropout_matches_oracle(cfg, path, tol, kw):
    """Hidden activations and their gradient are multiplied by keep / (1 - rate); the mask is a seeded input."""
    _check_layer(cfg, path, tol, dropout=0.4, d_aux=0.7, **kw)
