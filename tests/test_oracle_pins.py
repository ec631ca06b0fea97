"""Pins for the CPU oracle: each test checks oracle/switch_oracle.py against something other than itself.

What the paper and the mathematics fix: Eq. 3 values, a hand-worked example, a literal one-hot
dispatch/combine formulation (the appendix pseudo-code's data flow, rebuilt here with dense tensors),
brute-force position counting, the E = 1 reduction to a dense FFN, the closed forms of the auxiliary
loss, constructed routings with a known answer, and central finite differences for the backward pass.
"""
import json
import math
import os

import numpy as np
import pytest

from oracle import switch_oracle as so

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_layer(T, d, f, E, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((T, d))
    W_r = rng.standard_normal((d, E)) * scale / math.sqrt(d)
    W_in = rng.standard_normal((E, d, f)) / math.sqrt(d)
    W_out = rng.standard_normal((E, f, d)) / math.sqrt(f)
    return x, W_r, W_in, W_out


# ------------------------------------------------------------------ Eq. 3
def test_capacity_matches_eq3_table():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "capacity_eq3.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) >= 5
    for T, E, cf, C in rows:
        assert so.expert_capacity(int(T), int(E), float(cf)) == int(C)


def test_capacity_floor_and_cap():
    assert so.expert_capacity(10, 4, 1.0) == 2          # 2.5 floored
    assert so.expert_capacity(10, 4, 1.25) == 3         # 3.125 floored
    assert so.expert_capacity(8, 1, 2.0) == 8           # never more slots than tokens


# ------------------------------------------------------------------ hand-worked example
def test_hand_worked_example():
    g = json.load(open(os.path.join(GOLDEN, "hand_example.json")))
    W_r = np.array(g["W_r_times_1_over_ln3"], dtype=float) * math.log(3.0)
    out = so.switch_forward(np.array(g["x"], float), W_r, np.array(g["W_in"], float), np.array(g["W_out"], float),
                            g["capacity_factor"], g["alpha"])
    ex = g["expect"]
    np.testing.assert_allclose(out["p"], ex["p"], rtol=0, atol=1e-14)
    assert out["e"].tolist() == ex["e"]
    np.testing.assert_allclose(out["g"], ex["g"], atol=1e-14)
    assert out["C"] == ex["C"]
    assert out["pos"].tolist() == ex["pos"]
    assert out["keep"].astype(int).tolist() == ex["keep"]
    assert out["slot"].tolist() == ex["slot"]
    assert out["count"].tolist() == ex["count"]
    assert out["kept"].tolist() == ex["kept"]
    np.testing.assert_allclose(out["y"], ex["y"], atol=1e-13)
    np.testing.assert_allclose(out["f"], ex["f"], atol=1e-15)
    np.testing.assert_allclose(out["P"], ex["P"], atol=1e-14)
    assert abs(out["aux"] - ex["aux"]) < 1e-15


# ------------------------------------------------------------------ softmax / gate
def test_softmax_rows_sum_to_one_and_gate_bounds():
    x, W_r, _, _ = _rand_layer(200, 16, 8, 12, seed=1, scale=3.0)
    p = so.router_probs(so.router_logits(x, W_r))
    np.testing.assert_allclose(p.sum(1), 1.0, atol=1e-14)
    e, g = so.top1(p)
    assert np.all(g >= 1.0 / 12 - 1e-15) and np.all(g <= 1.0)
    assert np.all(p[np.arange(200), e] == p.max(1))


def test_softmax_against_direct_formula_and_shift_invariance():
    rng = np.random.default_rng(2)
    h = rng.standard_normal((7, 5))
    direct = np.array([[math.exp(h[t, i]) / sum(math.exp(h[t, j]) for j in range(5)) for i in range(5)]
                       for t in range(7)])
    np.testing.assert_allclose(so.router_probs(h), direct, rtol=1e-14)
    np.testing.assert_allclose(so.router_probs(h + 1000.0), direct, rtol=1e-12)   # no overflow, same value


def test_logits_orientation_and_bias():
    # h[t, i] = sum_k x[t, k] W_r[k, i] (+ b_i): a transposed operand or dropped bias changes these numbers.
    x = np.array([[1.0, 2.0, 3.0]])
    W_r = np.array([[1.0, 0.0], [0.0, 10.0], [100.0, 0.0]])
    np.testing.assert_array_equal(so.router_logits(x, W_r), [[301.0, 20.0]])
    np.testing.assert_array_equal(so.router_logits(x, W_r, np.array([0.5, -1.0])), [[301.5, 19.0]])


def test_argmax_tie_goes_to_lowest_index():
    p = np.array([[0.4, 0.4, 0.2], [0.1, 0.45, 0.45]])
    e, g = so.top1(p)
    assert e.tolist() == [0, 1] and g.tolist() == [0.4, 0.45]


# ------------------------------------------------------------------ dispatch plan
def _brute_force_plan(e, E, C):
    T = len(e)
    pos = [sum(1 for s in range(t) if e[s] == e[t]) for t in range(T)]          # O(T^2) definition
    keep = [pos[t] < C for t in range(T)]
    slot = [e[t] * C + pos[t] if keep[t] else -1 for t in range(T)]
    tos = [-1] * (E * C)
    for t in range(T):
        if keep[t]:
            tos[slot[t]] = t
    count = [sum(1 for t in range(T) if e[t] == i) for i in range(E)]
    return pos, keep, slot, tos, count


@pytest.mark.parametrize("T,E,C,seed", [(97, 5, 11, 0), (64, 8, 8, 1), (200, 3, 50, 2), (33, 7, 1, 3)])
def test_dispatch_plan_matches_brute_force(T, E, C, seed):
    rng = np.random.default_rng(seed)
    e = rng.integers(0, E, size=T)
    e[rng.random(T) < 0.4] = 0                      # skew so that expert 0 overflows
    plan = so.dispatch_plan(e, E, C)
    pos, keep, slot, tos, count = _brute_force_plan(e.tolist(), E, C)
    assert plan["pos"].tolist() == pos
    assert plan["keep"].tolist() == keep
    assert plan["slot"].tolist() == slot
    assert plan["token_of_slot"].tolist() == tos
    assert plan["count"].tolist() == count
    assert plan["kept"].tolist() == [min(c, C) for c in count]
    # invariants: kept slots of an expert are 0..kept-1 in increasing token order
    for i in range(E):
        toks = [t for t in plan["token_of_slot"][i * C:(i + 1) * C] if t >= 0]
        assert toks == sorted(toks) and len(toks) == plan["kept"][i]
        assert all(plan["token_of_slot"][i * C + j] >= 0 for j in range(plan["kept"][i]))
    assert plan["kept"].sum() <= min(T, E * C)


def test_round_robin_routing_has_no_drops_and_uniform_f():
    # x_t = c * unit(t mod E), W_r = identity block  =>  e_t = t mod E, pos_t = floor(t / E), nothing dropped at cf = 1
    T, E, d = 64, 8, 8
    x = np.zeros((T, d))
    x[np.arange(T), np.arange(T) % E] = 5.0
    W_r = np.eye(d, E)
    W_in = np.ones((E, d, 4))
    W_out = np.ones((E, 4, d))
    out = so.switch_forward(x, W_r, W_in, W_out, 1.0, 0.01)
    assert out["e"].tolist() == [t % E for t in range(T)]
    assert out["pos"].tolist() == [t // E for t in range(T)]
    assert out["keep"].all() and out["C"] == 8
    assert abs(out["aux"] - 0.01) < 1e-15            # f uniform => aux = alpha whatever P is (sum P = 1)


def test_zero_router_sends_everything_to_expert_zero():
    T, E, d, f = 40, 4, 6, 5
    x, _, W_in, W_out = _rand_layer(T, d, f, E, seed=3)
    out = so.switch_forward(x, np.zeros((d, E)), W_in, W_out, 1.0, 0.01)
    C = out["C"]
    assert C == 10 and (out["e"] == 0).all()
    assert out["keep"].tolist() == [t < C for t in range(T)]         # exactly the first C tokens are kept
    np.testing.assert_allclose(out["g"], 0.25)
    assert abs(out["aux"] - 0.01) < 1e-15            # P uniform => aux = alpha whatever f is (sum f = 1)
    assert np.all(out["y"][C:] == 0.0)               # dropped tokens: no computation, zero rows
    dense = np.maximum(x[:C] @ W_in[0], 0) @ W_out[0]
    np.testing.assert_allclose(out["y"][:C], 0.25 * dense, rtol=1e-13)


def test_aux_loss_upper_bound_and_definition():
    x, W_r, W_in, W_out = _rand_layer(128, 8, 4, 6, seed=4, scale=4.0)
    out = so.switch_forward(x, W_r, W_in, W_out, 1.0, 0.03)
    T, E = 128, 6
    # Eq. 4-6 written as explicit loops
    f = [sum(1 for t in range(T) if out["e"][t] == i) / T for i in range(E)]
    P = [sum(out["p"][t, i] for t in range(T)) / T for i in range(E)]
    assert abs(out["aux"] - 0.03 * E * sum(fi * Pi for fi, Pi in zip(f, P))) < 1e-15
    assert out["aux"] <= 0.03 * E + 1e-15
    assert abs(sum(f) - 1) < 1e-15 and abs(sum(P) - 1) < 1e-14
    # f is counted before the capacity cut: it does not change when the capacity shrinks
    out_small = so.switch_forward(x, W_r, W_in, W_out, 0.25, 0.03)
    assert not out_small["keep"].all()
    assert out_small["aux"] == out["aux"]


# ------------------------------------------------------------------ whole forward
def test_single_expert_reduces_to_dense_ffn():
    T, d, f = 24, 10, 14
    x, W_r, W_in, W_out = _rand_layer(T, d, f, 1, seed=5)
    out = so.switch_forward(x, W_r, W_in, W_out, 1.0, 0.01)
    np.testing.assert_allclose(out["g"], 1.0, atol=0)
    np.testing.assert_allclose(out["y"], np.maximum(x @ W_in[0], 0) @ W_out[0], rtol=1e-13)
    assert abs(out["aux"] - 0.01) < 1e-16
    half = so.switch_forward(x, W_r, W_in, W_out, 0.5, 0.01)     # capacity 12: first 12 rows, rest zero
    np.testing.assert_allclose(half["y"][:12], out["y"][:12], rtol=1e-13)
    assert np.all(half["y"][12:] == 0)


def _literal_one_hot_layer(x, W_r, W_in, W_out, cf, alpha):
    """The layer as dense one-hot dispatch / combine tensors and einsums (the appendix's data flow)."""
    T, d = x.shape
    E = W_r.shape[1]
    C = int(math.floor(T * cf / E))
    logits = np.einsum("td,de->te", x, W_r)
    probs = np.exp(logits - logits.max(1, keepdims=True))
    probs /= probs.sum(1, keepdims=True)
    index = probs.argmax(1)
    gate = probs.max(1)
    mask = np.eye(E)[index]                                        # [T, E] one-hot
    density = mask.mean(0)
    density_proxy = probs.mean(0)
    aux = alpha * np.mean(density * density_proxy) * E * E
    position = (np.cumsum(mask, axis=0) - 1.0) * mask              # 0-based position inside the expert
    mask = mask * (position < C)
    mask_flat = mask.sum(1)
    gate = gate * mask_flat
    pos_index = position.sum(1).astype(int)
    pos_one_hot = np.zeros((T, C))
    ok = pos_index < C
    pos_one_hot[np.flatnonzero(ok), pos_index[ok]] = 1.0
    combine = gate[:, None, None] * mask[:, :, None] * pos_one_hot[:, None, :]    # [T, E, C]
    dispatch = (combine != 0).astype(float)
    expert_inputs = np.einsum("td,tec->ecd", x, dispatch)
    hidden = np.maximum(np.einsum("ecd,edf->ecf", expert_inputs, W_in), 0.0)
    expert_outputs = np.einsum("ecf,efd->ecd", hidden, W_out)
    y = np.einsum("ecd,tec->td", expert_outputs, combine)
    return y, aux, dispatch


@pytest.mark.parametrize("T,d,f,E,cf,seed", [(48, 6, 10, 4, 1.0, 0), (64, 8, 12, 8, 1.25, 1), (40, 5, 7, 5, 0.5, 2)])
def test_index_formulation_equals_literal_one_hot_formulation(T, d, f, E, cf, seed):
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=seed, scale=2.0)
    out = so.switch_forward(x, W_r, W_in, W_out, cf, 0.01)
    y, aux, dispatch = _literal_one_hot_layer(x, W_r, W_in, W_out, cf, 0.01)
    np.testing.assert_allclose(out["y"], y, rtol=1e-12, atol=1e-13)
    assert abs(out["aux"] - aux) < 1e-15
    C = out["C"]
    mine = np.zeros((T, E, C))
    for t in range(T):
        if out["keep"][t]:
            mine[t, out["e"][t], out["pos"][t]] = 1.0
    np.testing.assert_array_equal(mine, dispatch)


def test_large_capacity_is_plain_top1_mixture():
    T, d, f, E = 50, 6, 9, 5
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=6, scale=2.0)
    out = so.switch_forward(x, W_r, W_in, W_out, float(E), 0.01)       # capacity = T: nothing can drop
    assert out["keep"].all()
    for t in range(T):
        i = out["e"][t]
        ref = out["p"][t, i] * (np.maximum(x[t] @ W_in[i], 0) @ W_out[i])
        np.testing.assert_allclose(out["y"][t], ref, rtol=1e-12, atol=1e-14)


def test_expert_subset_restricts_only_ffn_work():
    x, W_r, W_in, W_out = _rand_layer(60, 6, 8, 4, seed=7, scale=2.0)
    full = so.switch_forward(x, W_r, W_in, W_out, 1.0, 0.01)
    part = so.switch_forward(x, W_r, W_in, W_out, 1.0, 0.01, experts=[1, 3])
    sel = np.isin(full["e"], [1, 3])
    np.testing.assert_array_equal(part["y"][sel], full["y"][sel])
    assert np.all(part["y"][~sel] == 0)
    assert part["aux"] == full["aux"] and part["slot"].tolist() == full["slot"].tolist()


# ------------------------------------------------------------------ backward
def _loss(x, W_r, b, W_in, W_out, cf, alpha, R, d_aux, expert_index):
    out = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, router_bias=b, expert_index=expert_index)
    return float(np.sum(out["y"] * R) + d_aux * out["aux"])


def test_backward_matches_central_finite_differences():
    T, d, f, E, cf, alpha, d_aux = 16, 8, 16, 4, 0.75, 0.05, 1.7
    rng = np.random.default_rng(11)
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=11, scale=2.0)
    b = rng.standard_normal(E) * 0.3
    R = rng.standard_normal((T, d))
    fwd = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, router_bias=b)
    assert (~fwd["keep"]).sum() >= 2                       # some tokens are dropped in this case
    srt = np.sort(fwd["p"], axis=1)
    assert (srt[:, -1] - srt[:, -2]).min() > 1e-3          # no argmax boundary within reach of the step
    bwd = so.switch_backward(fwd, x, W_r, W_in, W_out, R, d_aux=d_aux)
    e_frozen = fwd["e"]
    eps = 1e-6

    def fd(arr, idx):
        old = arr[idx]
        arr[idx] = old + eps
        lp = _loss(x, W_r, b, W_in, W_out, cf, alpha, R, d_aux, e_frozen)
        arr[idx] = old - eps
        lm = _loss(x, W_r, b, W_in, W_out, cf, alpha, R, d_aux, e_frozen)
        arr[idx] = old
        return (lp - lm) / (2 * eps)

    for name, arr, grad in [("dx", x, bwd["dx"]), ("dW_r", W_r, bwd["dW_r"]), ("db", b, bwd["db"])]:
        num = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            num[idx] = fd(arr, idx)
        err = np.linalg.norm(num - grad) / np.linalg.norm(grad)
        assert err < 1e-7, (name, err)
    dW_in = np.stack([bwd["dW_in"][i] for i in range(E)])
    dW_out = np.stack([bwd["dW_out"][i] for i in range(E)])
    for name, arr, grad in [("dW_in", W_in, dW_in), ("dW_out", W_out, dW_out)]:
        idxs = [tuple(rng.integers(0, s) for s in arr.shape) for _ in range(150)]
        num = np.array([fd(arr, i) for i in idxs])
        ana = np.array([grad[i] for i in idxs])
        assert np.linalg.norm(num - ana) / np.linalg.norm(ana) < 1e-7, name


def test_backward_invariants():
    T, d, f, E = 40, 6, 8, 5
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=12, scale=3.0)
    rng = np.random.default_rng(12)
    dy = rng.standard_normal((T, d))
    # make expert 4 unreachable (huge negative bias) so that it has no tokens
    b = np.array([0.0, 0.0, 0.0, 0.0, -50.0])
    fwd = so.switch_forward(x, W_r, W_in, W_out, 0.5, 0.0, router_bias=b)       # alpha = 0
    assert fwd["count"][4] == 0 and (~fwd["keep"]).any()
    bwd = so.switch_backward(fwd, x, W_r, W_in, W_out, dy)
    np.testing.assert_allclose(bwd["dh"].sum(1), 0.0, atol=1e-14)            # softmax gradient sums to zero per token
    assert np.all(bwd["dx"][~fwd["keep"]] == 0.0)                            # dropped token, alpha = 0: no gradient at all
    assert np.all(bwd["dgate"][~fwd["keep"]] == 0.0)
    assert np.all(bwd["dW_in"][4] == 0) and np.all(bwd["dW_out"][4] == 0)    # expert without tokens
    # with alpha > 0 a dropped token still gets the auxiliary-loss gradient through P
    fwd2 = so.switch_forward(x, W_r, W_in, W_out, 0.5, 0.1, router_bias=b)
    bwd2 = so.switch_backward(fwd2, x, W_r, W_in, W_out, dy)
    assert np.abs(bwd2["dx"][~fwd2["keep"]]).max() > 0


def test_single_expert_backward_is_dense_ffn_backward():
    T, d, f = 12, 5, 7
    x, W_r, W_in, W_out = _rand_layer(T, d, f, 1, seed=13)
    dy = np.random.default_rng(13).standard_normal((T, d))
    fwd = so.switch_forward(x, W_r, W_in, W_out, 1.0, 0.01)
    bwd = so.switch_backward(fwd, x, W_r, W_in, W_out, dy)
    u = x @ W_in[0]
    a = np.maximum(u, 0)
    da = dy @ W_out[0].T
    du = da * (u > 0)
    np.testing.assert_allclose(bwd["dW_out"][0], a.T @ dy, rtol=1e-12)
    np.testing.assert_allclose(bwd["dW_in"][0], x.T @ du, rtol=1e-12)
    np.testing.assert_allclose(bwd["dx"], du @ W_in[0].T, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(bwd["dW_r"], 0.0, atol=1e-14)                 # p == 1 identically


def test_router_backward_helper_agrees_with_full_backward():
    T, d, f, E = 30, 6, 8, 4
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=14, scale=2.0)
    dy = np.random.default_rng(14).standard_normal((T, d))
    fwd = so.switch_forward(x, W_r, W_in, W_out, 0.75, 0.02)
    bwd = so.switch_backward(fwd, x, W_r, W_in, W_out, dy, d_aux=0.5)
    rb = so.router_backward_given_dgate(fwd["p"], fwd["e"], fwd["keep"], fwd["count"], bwd["dgate"], x, W_r,
                                        0.02, d_aux=0.5)
    np.testing.assert_allclose(rb["dW_r"], bwd["dW_r"], rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(rb["dx_router"], bwd["dx_router"], rtol=1e-13, atol=1e-15)


# ------------------------------------------------------------------ residual connection around the layer (Fig. 2, Section 2.2)
def test_residual_output_is_input_plus_layer_and_dropped_rows_pass_through():
    T, d, f, E = 40, 6, 8, 4
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=21, scale=2.0)
    plain = so.switch_forward(x, W_r, W_in, W_out, 0.5, 0.01)
    res = so.switch_forward(x, W_r, W_in, W_out, 0.5, 0.01, residual=True)
    dropped = ~res["keep"]
    assert dropped.sum() >= 3
    assert np.array_equal(res["y"][dropped], x[dropped])                    # a dropped token leaves the layer unchanged
    assert np.array_equal(res["layer_y"], plain["y"])
    np.testing.assert_allclose(res["y"] - x, plain["y"], rtol=0, atol=1e-15)
    assert res["aux"] == plain["aux"] and res["slot"].tolist() == plain["slot"].tolist()


def test_residual_backward_adds_dy_and_matches_finite_differences():
    T, d, f, E, cf, alpha, d_aux = 14, 5, 9, 3, 0.75, 0.03, 0.9
    rng = np.random.default_rng(22)
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=22, scale=2.0)
    R = rng.standard_normal((T, d))
    fwd = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, residual=True)
    srt = np.sort(fwd["p"], axis=1)
    assert (srt[:, -1] - srt[:, -2]).min() > 1e-3 and (~fwd["keep"]).any()
    bwd = so.switch_backward(fwd, x, W_r, W_in, W_out, R, d_aux=d_aux)
    plain_fwd = so.switch_forward(x, W_r, W_in, W_out, cf, alpha)
    plain = so.switch_backward(plain_fwd, x, W_r, W_in, W_out, R, d_aux=d_aux)
    np.testing.assert_allclose(bwd["dx"], plain["dx"] + R, rtol=0, atol=1e-14)   # the skip path carries dy unchanged
    for k in ("dW_r", "dgate"):
        assert np.array_equal(bwd[k], plain[k])                              # no other gradient sees the skip path
    e_frozen, eps = fwd["e"], 1e-6

    def loss():
        out = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, expert_index=e_frozen, residual=True)
        return float(np.sum(out["y"] * R) + d_aux * out["aux"])

    num = np.zeros_like(x)
    for idx in np.ndindex(x.shape):
        old = x[idx]
        x[idx] = old + eps
        lp = loss()
        x[idx] = old - eps
        lm = loss()
        x[idx] = old
        num[idx] = (lp - lm) / (2 * eps)
    assert np.linalg.norm(num - bwd["dx"]) / np.linalg.norm(bwd["dx"]) < 1e-7


# ------------------------------------------------------------------ several routing groups (the pseudo-code's [num_cores] dimension)
def _literal_grouped_layer(x, W_r, W_in, W_out, cf, alpha, G):
    """The appendix formulation with its leading group dimension: tensors [G, T/G, ...], one-hot dispatch and
    combine tensors [G, T/G, E, C], experts shared; loss = mean(density . density_proxy) . E^2."""
    T, d = x.shape
    n = T // G
    E = W_r.shape[1]
    C = int(math.floor(n * cf / E))
    xg = x.reshape(G, n, d)
    logits = np.einsum("gtd,de->gte", xg, W_r)
    probs = np.exp(logits - logits.max(2, keepdims=True))
    probs /= probs.sum(2, keepdims=True)
    index = probs.argmax(2)
    gate = probs.max(2)
    mask = np.eye(E)[index]                                            # [G, n, E]
    aux = alpha * np.mean(mask.mean(1) * probs.mean(1)) * E * E
    position = (np.cumsum(mask, axis=1) - 1.0) * mask
    mask = mask * (position < C)
    gate = gate * mask.sum(2)
    pos_index = position.sum(2).astype(int)
    pos_one_hot = (np.arange(C)[None, None, :] == pos_index[:, :, None]).astype(float)
    combine = gate[..., None, None] * mask[..., None] * pos_one_hot[:, :, None, :]   # [G, n, E, C]
    dispatch = (combine != 0).astype(float)
    expert_inputs = np.einsum("gtd,gtec->egcd", xg, dispatch)
    hidden = np.maximum(np.einsum("egcd,edf->egcf", expert_inputs, W_in), 0.0)
    expert_outputs = np.einsum("egcf,efd->egcd", hidden, W_out)
    y = np.einsum("egcd,gtec->gtd", expert_outputs, combine)
    return y.reshape(T, d), aux, dispatch


@pytest.mark.parametrize("T,d,f,E,cf,G,seed", [(48, 6, 10, 4, 1.0, 3, 0), (64, 8, 12, 8, 1.25, 2, 1), (60, 5, 7, 5, 0.5, 4, 2)])
def test_grouped_layer_equals_literal_formulation_with_group_dimension(T, d, f, E, cf, G, seed):
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=seed, scale=2.0)
    out = so.switch_forward_groups(x, W_r, W_in, W_out, cf, 0.01, G)
    y, aux, dispatch = _literal_grouped_layer(x, W_r, W_in, W_out, cf, 0.01, G)
    np.testing.assert_allclose(out["y"], y, rtol=1e-12, atol=1e-13)
    assert abs(out["aux"] - aux) < 1e-15
    n, C = T // G, out["C"]
    mine = np.zeros((G, n, E, C))
    for t in range(T):
        if out["keep"][t]:
            mine[t // n, t % n, out["e"][t], out["pos"][t]] = 1.0
    np.testing.assert_array_equal(mine, dispatch)
    # merged plan: a permutation of the kept tokens, expert-major, groups in order, token order inside a group
    kept_tok = np.flatnonzero(out["keep"])
    order = sorted(kept_tok, key=lambda t: (out["e"][t], t))
    rows = [s for s in out["token_of_slot"] if s >= 0]
    assert rows == order
    for i in range(E):
        seg = out["token_of_slot"][i * G * C:(i + 1) * G * C]
        k = int(out["kept"][i])
        assert np.all(seg[:k] >= 0) and np.all(seg[k:] == -1)           # an expert's rows are dense from its first row
    assert np.array_equal(out["slot"][kept_tok], [int(np.flatnonzero(out["token_of_slot"] == t)[0]) for t in kept_tok])


def test_one_group_is_the_plain_layer_and_groups_do_not_share_capacity():
    T, d, f, E = 64, 6, 8, 4
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=31, scale=2.0)
    one = so.switch_forward_groups(x, W_r, W_in, W_out, 0.75, 0.02, 1)
    plain = so.switch_forward(x, W_r, W_in, W_out, 0.75, 0.02)
    assert np.array_equal(one["y"], plain["y"]) and one["aux"] == plain["aux"]
    assert np.array_equal(one["slot"], plain["slot"])
    two = so.switch_forward_groups(x, W_r, W_in, W_out, 0.75, 0.02, 2)
    assert two["C"] == plain["C"] // 2
    # an expert that overflows in group 0 drops tokens there even if group 1 leaves room
    assert np.all(two["kept_g"] <= two["C"]) and (two["count_g"] > two["C"]).any()


def test_grouped_backward_matches_finite_differences():
    T, d, f, E, cf, alpha, d_aux, G = 16, 5, 7, 3, 0.75, 0.04, 1.3, 2
    rng = np.random.default_rng(32)
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=32, scale=2.0)
    R = rng.standard_normal((T, d))
    fwd = so.switch_forward_groups(x, W_r, W_in, W_out, cf, alpha, G)
    srt = np.sort(fwd["p"], axis=1)
    assert (srt[:, -1] - srt[:, -2]).min() > 1e-3 and (~fwd["keep"]).any()
    bwd = so.switch_backward_groups(fwd, x, W_r, W_in, W_out, R, d_aux=d_aux)
    e_frozen, eps = fwd["e"], 1e-6

    def loss():
        out = so.switch_forward_groups(x, W_r, W_in, W_out, cf, alpha, G, expert_index=e_frozen)
        return float(np.sum(out["y"] * R) + d_aux * out["aux"])

    def fd(arr, idx):
        old = arr[idx]
        arr[idx] = old + eps
        lp = loss()
        arr[idx] = old - eps
        lm = loss()
        arr[idx] = old
        return (lp - lm) / (2 * eps)

    dW_in = np.stack([bwd["dW_in"][i] for i in range(E)])
    dW_out = np.stack([bwd["dW_out"][i] for i in range(E)])
    for name, arr, grad in [("dx", x, bwd["dx"]), ("dW_r", W_r, bwd["dW_r"]), ("dW_in", W_in, dW_in),
                            ("dW_out", W_out, dW_out)]:
        idxs = list(np.ndindex(arr.shape))
        if len(idxs) > 200:
            idxs = [idxs[i] for i in rng.choice(len(idxs), 200, replace=False)]
        num = np.array([fd(arr, i) for i in idxs])
        ana = np.array([grad[i] for i in idxs])
        assert np.linalg.norm(num - ana) / np.linalg.norm(ana) < 1e-7, name


# ------------------------------------------------------------------ No-Token-Left-Behind, stage 2 (Appendix B)
def test_reroute_hand_example():
    # 6 tokens, 3 experts, capacity 2.  First choices 0 0 0 0 1 2 -> tokens 2, 3 overflow expert 0.  Second choices of
    # tokens 2 and 3 are experts 1 and 1: expert 1 has one slot left after its own token 4, so token 2 gets it
    # (token order) and token 3 stays dropped.
    p = np.array([[.7, .2, .1], [.6, .3, .1], [.5, .3, .2], [.5, .4, .1], [.1, .8, .1], [.2, .1, .7]])
    e, _ = so.top1(p)
    plan = so.dispatch_plan(e, 3, 2)
    alt = so.second_choice(p, e)
    assert alt.tolist() == [1, 1, 1, 1, 0, 0]
    out = so.reroute_overflow(plan, e, alt, 3, 2)
    assert out["keep"].tolist() == [True, True, True, False, True, True]
    assert out["e_proc"].tolist() == [0, 0, 1, 0, 1, 2]
    assert out["slot"].tolist() == [0, 1, 3, -1, 2, 4]
    assert out["kept"].tolist() == [2, 2, 1]
    assert out["token_of_slot"].tolist() == [0, 1, 4, 2, 5, -1]
    ties = np.array([[.4, .4, .2], [.2, .4, .4], [.5, .25, .25]])
    assert so.second_choice(ties, np.array([0, 1, 0])).tolist() == [1, 2, 1]     # ties: lowest index among the others


def _reroute_brute_force(p, E, C):
    """The figure's description, one token at a time: stage 1 for everybody, then stage 2 for the overflowed."""
    T = p.shape[0]
    order = np.argsort(-p, axis=1, kind="stable")
    load = [[] for _ in range(E)]
    dropped = []
    for t in range(T):
        (load[order[t, 0]].append(t) if len(load[order[t, 0]]) < C else dropped.append(t))
    for t in dropped:
        if len(load[order[t, 1]]) < C:
            load[order[t, 1]].append(t)
    return load


@pytest.mark.parametrize("T,E,cf,seed", [(60, 4, 0.75, 0), (80, 8, 1.0, 1), (33, 3, 0.5, 2), (64, 4, 4.0, 3)])
def test_reroute_matches_brute_force_and_keeps_stage_one(T, E, cf, seed):
    rng = np.random.default_rng(seed)
    p = so.router_probs(rng.standard_normal((T, E)) * 2.0 + np.linspace(1.5, 0.0, E))
    e, _ = so.top1(p)
    C = so.expert_capacity(T, E, cf)
    plan = so.dispatch_plan(e, E, C)
    out = so.reroute_overflow(plan, e, so.second_choice(p, e), E, C)
    load = _reroute_brute_force(p, E, C)
    for i in range(E):
        assert out["token_of_slot"][i * C:i * C + len(load[i])].tolist() == load[i]
        assert out["kept"][i] == len(load[i]) <= C
    assert np.array_equal(out["slot"][plan["keep"]], plan["slot"][plan["keep"]])       # stage 1 is untouched
    assert out["keep"].sum() >= plan["keep"].sum()
    if cf >= 4.0:
        assert np.array_equal(out["slot"], plan["slot"])                                # nothing overflowed


def test_reroute_layer_gate_and_gradient():
    T, d, f, E, cf, alpha, d_aux = 18, 5, 8, 3, 0.67, 0.03, 1.1
    rng = np.random.default_rng(41)
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=41, scale=2.0)
    b = np.array([1.0, 0.0, -0.5])                                       # expert 0 overflows
    R = rng.standard_normal((T, d))
    fwd = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, router_bias=b, reroute=True)
    plain = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, router_bias=b)
    moved = fwd["rerouted"]
    assert moved.sum() >= 2 and (~fwd["keep"]).sum() < (~plain["keep"]).sum()
    assert fwd["aux"] == plain["aux"]                                    # f still counts the argmax (Eq. 5)
    for t in np.flatnonzero(moved):                                      # Eq. 2 with the expert that processes the token
        i = fwd["e_proc"][t]
        want = fwd["p"][t, i] * (np.maximum(x[t] @ W_in[i], 0.0) @ W_out[i])
        np.testing.assert_allclose(fwd["y"][t], want, rtol=1e-12, atol=1e-14)
        assert i != fwd["e"][t] and fwd["p"][t, i] == np.sort(fwd["p"][t])[-2]
    stay = plain["keep"]
    np.testing.assert_array_equal(fwd["y"][stay], plain["y"][stay])
    # gradients against central differences with the routing frozen
    srt = np.sort(fwd["p"], axis=1)
    assert (srt[:, -1] - srt[:, -2]).min() > 1e-3 and (srt[:, -2] - srt[:, -3]).min() > 1e-3
    bwd = so.switch_backward(fwd, x, W_r, W_in, W_out, R, d_aux=d_aux)
    e_frozen, alt_frozen, eps = fwd["e"], fwd["alt"], 1e-6

    def loss():
        out = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, router_bias=b, expert_index=e_frozen, reroute=True,
                                alt_index=alt_frozen)
        return float(np.sum(out["y"] * R) + d_aux * out["aux"])

    for name, arr, grad in [("dx", x, bwd["dx"]), ("dW_r", W_r, bwd["dW_r"])]:
        num = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            old = arr[idx]
            arr[idx] = old + eps
            lp = loss()
            arr[idx] = old - eps
            lm = loss()
            arr[idx] = old
            num[idx] = (lp - lm) / (2 * eps)
        assert np.linalg.norm(num - grad) / np.linalg.norm(grad) < 1e-7, name


# ------------------------------------------------------------------ No-Token-Left-Behind, iterated (Appendix B, figure caption)
def test_next_choice_walks_every_expert_once_in_order_of_probability():
    rng = np.random.default_rng(61)
    p = so.router_probs(rng.standard_normal((40, 7)) * 2.0)
    p[3, 2] = p[3, 5]                                                    # an exact tie: the lower index comes first
    p[9] = 1.0 / 7                                                       # all equal: the ranking is 0, 1, .., 6
    e, _ = so.top1(p)
    np.testing.assert_array_equal(so.next_choice(p, e), so.second_choice(p, e))
    seen, prev = [e], e
    for _ in range(6):
        prev = so.next_choice(p, prev)
        seen.append(prev)
    seen = np.stack(seen, axis=1)                                        # [T, E]: the whole ranking
    assert np.array_equal(np.sort(seen, axis=1), np.tile(np.arange(7), (40, 1)))
    ranked = np.take_along_axis(p, seen, axis=1)
    assert (np.diff(ranked, axis=1) <= 0).all()
    assert seen[9].tolist() == list(range(7))
    i2, i5 = seen[3].tolist().index(2), seen[3].tolist().index(5)
    assert i5 == i2 + 1
    assert (so.next_choice(p, prev) == -1).all()                         # nothing after the last
    assert (so.next_choice(p, np.full(40, -1)) == -1).all()
    hand = np.array([[.1, .4, .2, .3]])
    assert [int(so.next_choice(hand, np.array([k]))[0]) for k in (1, 3, 2, 0)] == [3, 2, 0, -1]


def _iterated_reroute_brute_force(p, E, C, stages):
    """Stage 1 for everybody; then, stage after stage, the tokens still without a slot try the next expert of their
    own ranking, in token order (written with preference lists and plain Python lists)."""
    T = p.shape[0]
    prefs = [sorted(range(E), key=lambda i: (-p[t, i], i)) for t in range(T)]
    load = [[] for _ in range(E)]
    waiting = list(range(T))
    for s in range(stages + 1):
        still = []
        for t in waiting:
            i = prefs[t][s] if s < E else None
            if i is not None and len(load[i]) < C:
                load[i].append(t)
            else:
                still.append(t)
        waiting = still
    return load, waiting


@pytest.mark.parametrize("T,E,cf,stages,seed", [(60, 4, 0.75, 2, 0), (80, 8, 1.0, 3, 1), (33, 3, 0.5, 2, 2),
                                                (90, 6, 1.0, 5, 3), (50, 5, 0.6, 4, 4), (40, 4, 1.0, 6, 5)])
def test_iterated_reroute_matches_brute_force(T, E, cf, stages, seed):
    rng = np.random.default_rng(seed)
    p = so.router_probs(rng.standard_normal((T, E)) * 2.0 + np.linspace(2.5, 0.0, E))
    e, _ = so.top1(p)
    C = so.expert_capacity(T, E, cf)
    plan, prev, kept_before = so.dispatch_plan(e, E, C), e, None
    first = plan
    for s in range(stages):
        prev = so.next_choice(p, prev)
        before = plan
        plan = so.reroute_overflow(plan, e, prev, E, C)
        assert np.array_equal(plan["slot"][before["keep"]], before["slot"][before["keep"]])   # earlier stages untouched
        load, waiting = _iterated_reroute_brute_force(p, E, C, s + 1)
        for i in range(E):
            assert plan["token_of_slot"][i * C:i * C + len(load[i])].tolist() == load[i]
            assert plan["kept"][i] == len(load[i]) <= C
        assert np.flatnonzero(~plan["keep"]).tolist() == waiting
    assert np.array_equal(plan["rerouted"], plan["keep"] & ~first["keep"])
    assert np.array_equal(plan["e_proc"][first["keep"]], e[first["keep"]])
    moved = plan["rerouted"]
    assert np.array_equal(plan["slot"][moved] // C, plan["e_proc"][moved])
    if stages >= E - 1:                                                  # every token has tried every expert:
        assert plan["keep"].sum() == min(T, E * C)                       # a token is dropped only if all slots are taken


def test_iterated_reroute_in_the_layer_gate_and_gradient():
    T, d, f, E, cf, alpha, d_aux, stages = 20, 5, 8, 4, 0.8, 0.03, 1.1, 3
    rng = np.random.default_rng(43)
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=43, scale=2.0)
    b = np.array([1.5, 0.8, 0.0, -0.5])                                  # experts 0 and 1 overflow
    R = rng.standard_normal((T, d))
    one = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, router_bias=b, reroute=True)
    fwd = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, router_bias=b, reroute=True, reroute_stages=stages)
    assert fwd["keep"].sum() == min(T, E * fwd["C"]) > one["keep"].sum()          # E - 1 extra stages fill every slot
    assert fwd["aux"] == one["aux"]
    np.testing.assert_array_equal(fwd["y"][one["keep"]], one["y"][one["keep"]])   # stage 2's tokens stay where they were
    later = fwd["keep"] & ~one["keep"]
    assert later.sum() >= 1
    for t in np.flatnonzero(later):
        i = fwd["e_proc"][t]
        want = fwd["p"][t, i] * (np.maximum(x[t] @ W_in[i], 0.0) @ W_out[i])
        np.testing.assert_allclose(fwd["y"][t], want, rtol=1e-12, atol=1e-14)
        assert fwd["p"][t, i] <= np.sort(fwd["p"][t])[-3]                          # third choice or later
    assert fwd["alt"].shape == (stages, T)
    bwd = so.switch_backward(fwd, x, W_r, W_in, W_out, R, d_aux=d_aux)
    e_frozen, alt_frozen, eps = fwd["e"], fwd["alt"], 1e-6       # the routing is frozen: the loss is smooth in x, W_r

    def loss():
        out = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, router_bias=b, expert_index=e_frozen, reroute=True,
                                reroute_stages=stages, alt_index=alt_frozen)
        return float(np.sum(out["y"] * R) + d_aux * out["aux"])

    for name, arr, grad in [("dx", x, bwd["dx"]), ("dW_r", W_r, bwd["dW_r"])]:
        num = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            old = arr[idx]
            arr[idx] = old + eps
            lp = loss()
            arr[idx] = old - eps
            lm = loss()
            arr[idx] = old
            num[idx] = (lp - lm) / (2 * eps)
        assert np.linalg.norm(num - grad) / np.linalg.norm(grad) < 1e-7, name


# ------------------------------------------------------------------ exploration noise on the router logits (appendix pseudo-code)
def test_logit_noise_is_additive_and_its_mean_cancels_in_the_softmax():
    T, d, f, E = 24, 6, 8, 5
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=51, scale=2.0)
    rng = np.random.default_rng(51)
    eps = 0.3
    noise = rng.uniform(1 - eps, 1 + eps, size=(T, E))
    h0 = so.router_logits(x, W_r)
    np.testing.assert_allclose(so.router_logits(x, W_r, router_noise=noise), h0 + noise, rtol=0, atol=1e-15)
    # uniform(1 - eps, 1 + eps) = 1 + uniform(-eps, eps): the common 1 is a shift the softmax does not see
    p1 = so.router_probs(so.router_logits(x, W_r, router_noise=noise))
    p2 = so.router_probs(so.router_logits(x, W_r, router_noise=noise - 1.0))
    np.testing.assert_allclose(p1, p2, rtol=1e-13)
    a = so.switch_forward(x, W_r, W_in, W_out, 1.0, 0.01, router_noise=np.ones((T, E)))
    b = so.switch_forward(x, W_r, W_in, W_out, 1.0, 0.01)
    np.testing.assert_allclose(a["p"], b["p"], rtol=1e-13)
    assert np.array_equal(a["e"], b["e"]) and np.array_equal(a["slot"], b["slot"])
    # noise that large does move tokens, and the gradient treats it as a constant
    c = so.switch_forward(x, W_r, W_in, W_out, 1.0, 0.01, router_noise=noise * 5.0)
    assert (c["e"] != b["e"]).any()
    R = rng.standard_normal((T, d))
    bwd = so.switch_backward(c, x, W_r, W_in, W_out, R)
    srt = np.sort(c["p"], axis=1)
    assert (srt[:, -1] - srt[:, -2]).min() > 1e-4
    e_frozen, step = c["e"], 1e-6
    num = np.zeros_like(W_r)
    for idx in np.ndindex(W_r.shape):
        old = W_r[idx]
        vals = []
        for sgn in (1.0, -1.0):
            W_r[idx] = old + sgn * step
            out = so.switch_forward(x, W_r, W_in, W_out, 1.0, 0.01, router_noise=noise * 5.0, expert_index=e_frozen)
            vals.append(float(np.sum(out["y"] * R) + out["aux"]))
        W_r[idx] = old
        num[idx] = (vals[0] - vals[1]) / (2 * step)
    assert np.linalg.norm(num - bwd["dW_r"]) / np.linalg.norm(bwd["dW_r"]) < 1e-7


# ------------------------------------------------------------------ multiplicative jitter on the router's input (Appendix C, text)
def test_input_jitter_reaches_only_the_router_and_its_gradient_is_scaled():
    T, d, f, E, cf, alpha, d_aux = 14, 5, 7, 3, 1.0, 0.05, 0.8
    rng = np.random.default_rng(61)
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=61, scale=2.0)
    u = rng.uniform(0.7, 1.3, size=(T, d))
    fwd = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, router_jitter=u)
    np.testing.assert_allclose(fwd["h"], (x * u) @ W_r, rtol=1e-13)               # the router sees x . u
    for t in np.flatnonzero(fwd["keep"])[:5]:                                      # the experts see x
        i = fwd["e"][t]
        np.testing.assert_allclose(fwd["y"][t], fwd["g"][t] * (np.maximum(x[t] @ W_in[i], 0) @ W_out[i]), rtol=1e-12)
    same = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, router_jitter=np.ones((T, d)))
    plain = so.switch_forward(x, W_r, W_in, W_out, cf, alpha)
    assert np.array_equal(same["y"], plain["y"]) and same["aux"] == plain["aux"]
    # storage rounding is applied to the product only
    coarse = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, router_jitter=u, storage_round=lambda a: np.round(a, 1))
    np.testing.assert_allclose(coarse["h"], np.round(x * u, 1) @ W_r, rtol=1e-13)
    # gradients against central differences (routing frozen)
    R = rng.standard_normal((T, d))
    srt = np.sort(fwd["p"], axis=1)
    assert (srt[:, -1] - srt[:, -2]).min() > 1e-3
    bwd = so.switch_backward(fwd, x, W_r, W_in, W_out, R, d_aux=d_aux)
    e_frozen, eps = fwd["e"], 1e-6

    def loss():
        out = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, router_jitter=u, expert_index=e_frozen)
        return float(np.sum(out["y"] * R) + d_aux * out["aux"])

    for name, arr, grad in [("dx", x, bwd["dx"]), ("dW_r", W_r, bwd["dW_r"])]:
        num = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            old = arr[idx]
            arr[idx] = old + eps
            lp = loss()
            arr[idx] = old - eps
            lm = loss()
            arr[idx] = old
            num[idx] = (lp - lm) / (2 * eps)
        assert np.linalg.norm(num - grad) / np.linalg.norm(grad) < 1e-7, name


# ------------------------------------------------------------------ GEGLU experts (Table 9)
def test_gelu_closed_forms():
    from scipy.stats import norm
    z = np.linspace(-6, 6, 241)
    np.testing.assert_allclose(so.gelu(z), z * norm.cdf(z), rtol=1e-13, atol=1e-15)        # z . Phi(z)
    np.testing.assert_allclose(so.gelu(z) - so.gelu(-z), z, rtol=1e-13, atol=1e-15)        # odd part is z / 2 + z / 2
    assert so.gelu(0.0) == 0.0 and abs(so.gelu(10.0) - 10.0) < 1e-12 and abs(so.gelu(-10.0)) < 1e-12
    np.testing.assert_allclose(so.gelu_prime(z), norm.cdf(z) + z * norm.pdf(z), rtol=1e-12, atol=1e-15)
    h = 1e-6
    np.testing.assert_allclose(so.gelu_prime(z), (so.gelu(z + h) - so.gelu(z - h)) / (2 * h), rtol=1e-7, atol=1e-9)


def test_geglu_single_expert_is_the_dense_geglu_ffn_and_gradients_match_finite_differences():
    from scipy.stats import norm
    T, d, f = 10, 5, 6
    rng = np.random.default_rng(71)
    x = rng.standard_normal((T, d))
    W_r = rng.standard_normal((d, 1))
    W_in = rng.standard_normal((1, d, 2 * f)) * 0.7
    W_out = rng.standard_normal((1, f, d)) * 0.7
    out = so.switch_forward(x, W_r, W_in, W_out, 1.0, 0.01, geglu=True)
    a, b = x @ W_in[0][:, :f], x @ W_in[0][:, f:]
    np.testing.assert_allclose(out["y"], ((a * norm.cdf(a)) * b) @ W_out[0], rtol=1e-12)   # gate = 1 with one expert
    # several experts, drops, frozen routing: all gradients against central differences
    T, d, f, E, cf, alpha, d_aux = 16, 5, 6, 3, 0.75, 0.03, 1.2
    x = rng.standard_normal((T, d)) * 2
    W_r = rng.standard_normal((d, E))
    W_in = rng.standard_normal((E, d, 2 * f)) * 0.6
    W_out = rng.standard_normal((E, f, d)) * 0.6
    R = rng.standard_normal((T, d))
    fwd = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, geglu=True)
    srt = np.sort(fwd["p"], axis=1)
    assert (srt[:, -1] - srt[:, -2]).min() > 1e-3 and (~fwd["keep"]).any()
    bwd = so.switch_backward(fwd, x, W_r, W_in, W_out, R, d_aux=d_aux)
    e_frozen, eps = fwd["e"], 1e-6

    def loss():
        o = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, geglu=True, expert_index=e_frozen)
        return float(np.sum(o["y"] * R) + d_aux * o["aux"])

    dW_in = np.stack([bwd["dW_in"][i] for i in range(E)])
    dW_out = np.stack([bwd["dW_out"][i] for i in range(E)])
    for name, arr, grad in [("dx", x, bwd["dx"]), ("dW_r", W_r, bwd["dW_r"]), ("dW_in", W_in, dW_in),
                            ("dW_out", W_out, dW_out)]:
        idxs = list(np.ndindex(arr.shape))
        if len(idxs) > 150:
            idxs = [idxs[i] for i in rng.choice(len(idxs), 150, replace=False)]
        num = []
        for idx in idxs:
            old = arr[idx]
            arr[idx] = old + eps
            lp = loss()
            arr[idx] = old - eps
            lm = loss()
            arr[idx] = old
            num.append((lp - lm) / (2 * eps))
        ana = np.array([grad[i] for i in idxs])
        assert np.linalg.norm(np.array(num) - ana) / np.linalg.norm(ana) < 1e-7, name


# ------------------------------------------------------------------ top-2 routing (the Mixture-of-Experts comparator, Eq. 1-2)
def _literal_top2_layer(x, W_r, W_in, W_out, C):
    """Eq. 1-2 with the two highest-probability experts, one token at a time: first choices of all tokens are
    placed before any second choice; an assignment beyond the expert's capacity contributes nothing."""
    T, d = x.shape
    E = W_r.shape[1]
    logits = x @ W_r
    probs = np.exp(logits - logits.max(1, keepdims=True))
    probs /= probs.sum(1, keepdims=True)
    order = np.argsort(-probs, axis=1, kind="stable")
    load = np.zeros(E, dtype=int)
    y = np.zeros((T, d))
    placed = []
    for rnd in (0, 1):
        for t in range(T):
            i = order[t, rnd]
            if load[i] < C:
                load[i] += 1
                placed.append((rnd, t, i))
                y[t] += probs[t, i] * (np.maximum(x[t] @ W_in[i], 0.0) @ W_out[i])
    return y, placed, load


@pytest.mark.parametrize("T,d,f,E,cf,seed", [(40, 6, 9, 4, 2.0, 0), (48, 5, 8, 6, 1.0, 1), (30, 4, 6, 3, 0.5, 2)])
def test_top2_layer_equals_token_by_token_definition(T, d, f, E, cf, seed):
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=seed, scale=2.0)
    out = so.top2_forward(x, W_r, W_in, W_out, cf, 0.01)
    y, placed, load = _literal_top2_layer(x, W_r, W_in, W_out, out["C"])
    np.testing.assert_allclose(out["y"], y, rtol=1e-12, atol=1e-14)
    assert out["kept"].tolist() == load.tolist()
    assert sorted((v // T, v % T, int(out["e"][v])) for v in np.flatnonzero(out["keep"])) == sorted(placed)
    plain = so.switch_forward(x, W_r, W_in, W_out, cf, 0.01)
    assert out["aux"] == plain["aux"]                                        # f counts the first choice only
    assert np.array_equal(out["first"], plain["e"]) and np.all(out["second"] != out["first"])
    assert np.array_equal(out["slot"][:T][plain["keep"]], plain["slot"][plain["keep"]])   # round one is Switch routing
    if cf >= 2.0:
        assert out["keep"][:T].all()


def test_top2_with_the_skip_path_adds_the_input_and_passes_dy_through():
    """Fig. 2: the layer sits inside a residual connection.  With it the output is the plain output plus x (a token
    both of whose assignments overflowed comes out unchanged), and dx gains exactly dy."""
    T, d, f, E, cf = 24, 5, 7, 4, 0.5
    rng = np.random.default_rng(83)
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=83, scale=2.0)
    R = rng.standard_normal((T, d))
    plain = so.top2_forward(x, W_r, W_in, W_out, cf, 0.02)
    skip = so.top2_forward(x, W_r, W_in, W_out, cf, 0.02, residual=True)
    np.testing.assert_array_equal(skip["layer_y"], plain["y"])
    np.testing.assert_allclose(skip["y"] - x, plain["y"], rtol=0, atol=1e-14)
    lost = ~plain["keep"][:T] & ~plain["keep"][T:]
    assert lost.any()
    np.testing.assert_array_equal(skip["y"][lost], x[lost])
    b0 = so.top2_backward(plain, x, W_r, W_in, W_out, R)
    b1 = so.top2_backward(skip, x, W_r, W_in, W_out, R)
    np.testing.assert_allclose(b1["dx"], b0["dx"] + R, rtol=0, atol=1e-14)
    for k in ("dW_r", "dgate"):
        np.testing.assert_array_equal(b1[k], b0[k])


@pytest.mark.parametrize("residual", [False, True], ids=["plain", "skip"])
def test_top2_backward_matches_finite_differences(residual):
    T, d, f, E, cf, alpha, d_aux = 14, 5, 7, 4, 1.0, 0.04, 0.9
    rng = np.random.default_rng(81)
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=81, scale=2.0)
    R = rng.standard_normal((T, d))
    fwd = so.top2_forward(x, W_r, W_in, W_out, cf, alpha, residual=residual)
    srt = np.sort(fwd["p"], axis=1)
    assert (srt[:, -1] - srt[:, -2]).min() > 1e-3 and (srt[:, -2] - srt[:, -3]).min() > 1e-3 and (~fwd["keep"]).any()
    bwd = so.top2_backward(fwd, x, W_r, W_in, W_out, R, d_aux=d_aux)
    a, b, eps = fwd["first"], fwd["second"], 1e-6

    def loss():
        o = so.top2_forward(x, W_r, W_in, W_out, cf, alpha, first_index=a, second_index=b, residual=residual)
        return float(np.sum(o["y"] * R) + d_aux * o["aux"])

    dW_in = np.stack([bwd["dW_in"][i] for i in range(E)])
    dW_out = np.stack([bwd["dW_out"][i] for i in range(E)])
    for name, arr, grad in [("dx", x, bwd["dx"]), ("dW_r", W_r, bwd["dW_r"]), ("dW_in", W_in, dW_in),
                            ("dW_out", W_out, dW_out)]:
        idxs = list(np.ndindex(arr.shape))
        if len(idxs) > 150:
            idxs = [idxs[i] for i in rng.choice(len(idxs), 150, replace=False)]
        num = []
        for idx in idxs:
            old = arr[idx]
            arr[idx] = old + eps
            lp = loss()
            arr[idx] = old - eps
            lm = loss()
            arr[idx] = old
            num.append((lp - lm) / (2 * eps))
        ana = np.array([grad[i] for i in idxs])
        assert np.linalg.norm(np.array(num) - ana) / np.linalg.norm(ana) < 1e-7, name


# ------------------------------------------------------------------ expert dropout (fine-tuning regularisation)
def test_expert_dropout_scales_kept_hidden_units_and_gradients_match_finite_differences():
    T, d, f, E, cf, alpha, rate = 16, 5, 8, 3, 0.75, 0.03, 0.4
    rng = np.random.default_rng(91)
    x, W_r, W_in, W_out = _rand_layer(T, d, f, E, seed=91, scale=2.0)
    plain = so.switch_forward(x, W_r, W_in, W_out, cf, alpha)
    C = plain["C"]
    keep = rng.random((E * C, f)) >= rate
    fwd = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, expert_keep=keep, expert_dropout=rate)
    assert np.array_equal(fwd["slot"], plain["slot"]) and fwd["aux"] == plain["aux"]      # routing is untouched
    for t in np.flatnonzero(fwd["keep"])[:6]:
        i, s = fwd["e"][t], fwd["slot"][t]
        hidden = np.maximum(x[t] @ W_in[i], 0.0) * keep[s] / (1.0 - rate)
        np.testing.assert_allclose(fwd["y"][t], fwd["g"][t] * (hidden @ W_out[i]), rtol=1e-12, atol=1e-14)
    ones = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, expert_keep=np.ones((E * C, f), bool), expert_dropout=0.0)
    assert np.array_equal(ones["y"], plain["y"])
    R = rng.standard_normal((T, d))
    srt = np.sort(fwd["p"], axis=1)
    assert (srt[:, -1] - srt[:, -2]).min() > 1e-3
    bwd = so.switch_backward(fwd, x, W_r, W_in, W_out, R, d_aux=0.6)
    e_frozen, eps = fwd["e"], 1e-6

    def loss():
        o = so.switch_forward(x, W_r, W_in, W_out, cf, alpha, expert_index=e_frozen, expert_keep=keep, expert_dropout=rate)
        return float(np.sum(o["y"] * R) + 0.6 * o["aux"])

    dW_in = np.stack([bwd["dW_in"][i] for i in range(E)])
    dW_out = np.stack([bwd["dW_out"][i] for i in range(E)])
    for name, arr, grad in [("dx", x, bwd["dx"]), ("dW_r", W_r, bwd["dW_r"]), ("dW_in", W_in, dW_in),
                            ("dW_out", W_out, dW_out)]:
        idxs = list(np.ndindex(arr.shape))
        if len(idxs) > 150:
            idxs = [idxs[i] for i in rng.choice(len(idxs), 150, replace=False)]
        num = []
        for idx in idxs:
            old = arr[idx]
            arr[idx] = old + eps
            lp = loss()
            arr[idx] = old - eps
            lm = loss()
            arr[idx] = old
            num.append((lp - lm) / (2 * eps))
        ana = np.array([grad[i] for i in idxs])
        assert np.linalg.norm(np.array(num) - ana) / np.linalg.norm(ana) < 1e-7, name
