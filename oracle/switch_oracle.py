"""CPU oracle for one Switch FFN layer (Switch Transformer, arxiv 2101.03961): forward and backward.

TEST INFRASTRUCTURE, NOT THE PRODUCT.  This file is the slow, plain definition the CUDA library is
checked against.  Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may import
it; nothing in the product path does, and it shares no code with the CUDA path (it imports numpy only).

Everything is float64 and written in the paper's notation and order:
  h = x . W_r, p = softmax(h)                                   (Section 2.1, Eq. 1)
  top-1 expert e_t = argmax_i p_i(x_t), gate g_t = p_{e_t}(x_t)  (Section 2.1, "Switch Routing")
  expert capacity C = (tokens / experts) x capacity factor       (Section 2.2, Eq. 3)
  slots in token order, tokens beyond the capacity are dropped   (Section 2.2, Fig. 3; appendix router pseudo-code)
  auxiliary loss alpha . N . sum_i f_i P_i                       (Section 2.2, Eq. 4-6)
  expert FFN  y = ReLU(x W_in) W_out, no bias                    (Section 5, "Reviewing the FFN layer")
  layer output y_t = g_t . E_{e_t}(x_t)                          (Section 2.1, Eq. 2 with k = 1; Fig. 2)
The backward pass is the derivative of exactly those formulas (the paper leaves it to autodiff): the
gate keeps the router differentiable (Section 2.1), P is differentiable and f is not (Section 2.2).

Readings taken where the paper is silent or its listing is garbled (each is checked by a pin test):
  * capacity is floor(T * cf / E); positions are 0-based counts of earlier tokens with the same expert, and
    an expert keeps its first C tokens in token order (the listing's 1-based cumsum compared with `less`
    would keep C - 1, whereas Fig. 3 gives every expert a batch of exactly the capacity of Eq. 3);
  * f_i counts the argmax before the capacity cut (Eq. 5 is the argmax indicator);
  * argmax ties go to the lowest expert index;
  * a dropped token's output row is 0 (its gate is masked to 0); with `residual` the layer adds its own
    input, so a dropped token's row is exactly its input row;
  * the gate multiplies in full precision (no bfloat16 rounding of the combine weights);
  * one call is one routing group; the row order of x is the token order;
  * ReLU'(0) = 0;
  * an optional constant per-expert bias may be added to the logits (used by the overflow-stress
    workload only; the paper's router has none);
  * exploration noise follows the router pseudo-code (added to the logits), not the text's multiplicative
    jitter of the router input; it is passed in, never drawn here.

All functions here are pinned by tests/test_oracle_pins.py: none is "parity unpinned".
"""
from __future__ import annotations

import math

import numpy as np

F64 = np.float64


def expert_capacity(T: int, E: int, capacity_factor: float) -> int:
    """Eq. 3: expert capacity = (tokens per batch / number of experts) x capacity factor, floored, at most T."""
    C = int(math.floor(float(T) * float(capacity_factor) / float(E)))
    return min(C, T)


def router_logits(x, W_r, router_bias=None, router_noise=None):
    """Section 2.1: h(x) = W_r . x for every token; x [T, d], W_r [d, E] -> h [T, E] (float64).

    `router_noise` [T, E], when given, is added to the logits: the appendix's router pseudo-code adds
    uniform(1 - eps, 1 + eps) noise to the logits in training "for exploration across experts".  It is an input
    here (the caller draws it) and a constant of the backward pass."""
    h = np.asarray(x, dtype=F64) @ np.asarray(W_r, dtype=F64)
    if router_bias is not None:
        h = h + np.asarray(router_bias, dtype=F64)[None, :]
    if router_noise is not None:
        h = h + np.asarray(router_noise, dtype=F64)
    return h


def router_probs(h):
    """Eq. 1: p_i(x) = exp(h_i) / sum_j exp(h_j), evaluated with the row maximum subtracted."""
    z = h - h.max(axis=1, keepdims=True)
    ez = np.exp(z)
    return ez / ez.sum(axis=1, keepdims=True)


def top1(p):
    """Switch routing (k = 1): expert index e_t = argmax_i p[t, i] (lowest index on ties), gate g_t = p[t, e_t]."""
    e = np.argmax(p, axis=1).astype(np.int64)
    g = p[np.arange(p.shape[0]), e]
    return e, g


def load_balance_loss(p, e, alpha: float):
    """Eq. 4-6: alpha . N . sum_i f_i . P_i with f_i the argmax fraction and P_i the mean probability."""
    T, N = p.shape
    f = np.bincount(e, minlength=N).astype(F64) / T        # Eq. 5
    P = p.sum(axis=0) / T                                    # Eq. 6
    return float(alpha * N * np.dot(f, P)), f, P             # Eq. 4


def dispatch_plan(e, E: int, C: int):
    """Slot assignment in token order with the capacity cut (Section 2.2, Fig. 3).

    pos[t]  = number of earlier tokens routed to the same expert (0-based)
    keep[t] = pos[t] < C
    slot[t] = e[t] * C + pos[t] for kept tokens, -1 for dropped ones
    token_of_slot[s] = the token stored in slot s, -1 for an empty slot
    count[i] = tokens whose argmax is expert i (before the cut); kept[i] = min(count[i], C)
    """
    e = np.asarray(e, dtype=np.int64)
    T = e.shape[0]
    pos = np.zeros(T, dtype=np.int64)
    running = np.zeros(E, dtype=np.int64)
    for t in range(T):
        pos[t] = running[e[t]]
        running[e[t]] += 1
    count = running.copy()
    keep = pos < C
    slot = np.where(keep, e * C + pos, -1)
    token_of_slot = np.full(E * C, -1, dtype=np.int64)
    token_of_slot[slot[keep]] = np.flatnonzero(keep)
    kept = np.minimum(count, C)
    return {"pos": pos, "keep": keep, "slot": slot, "token_of_slot": token_of_slot, "count": count, "kept": kept}


def gelu(z):
    """GELU(z) = z . Phi(z) with Phi the standard normal distribution function (the exact form, not the tanh fit)."""
    z = np.asarray(z, dtype=F64)
    return z * 0.5 * (1.0 + _erf(z / math.sqrt(2.0)))


def gelu_prime(z):
    """d GELU / dz = Phi(z) + z . phi(z)."""
    z = np.asarray(z, dtype=F64)
    return 0.5 * (1.0 + _erf(z / math.sqrt(2.0))) + z * np.exp(-0.5 * z * z) / math.sqrt(2.0 * math.pi)


_erf = np.vectorize(math.erf, otypes=[F64])


def second_choice(p, e):
    """The expert with the second-highest probability of each token: the argmax over the experts other than e_t
    (lowest index on ties)."""
    q = np.array(p, dtype=F64, copy=True)
    q[np.arange(q.shape[0]), e] = -np.inf
    return np.argmax(q, axis=1).astype(np.int64)


def next_choice(p, prev):
    """The expert that follows prev[t] in token t's ranking of the experts: by probability, highest first, equal
    probabilities by index, lowest first.  From the argmax this is the second choice, from there the third, and so
    on; -1 once prev[t] was the last expert of the ranking (or is itself -1)."""
    p = np.asarray(p, dtype=F64)
    prev = np.asarray(prev, dtype=np.int64)
    T, E = p.shape
    out = np.full(T, -1, dtype=np.int64)
    for t in range(T):
        if prev[t] < 0:
            continue
        ranking = sorted(range(E), key=lambda i: (-p[t, i], i))
        place = ranking.index(int(prev[t]))
        if place + 1 < E:
            out[t] = ranking[place + 1]
    return out


def reroute_overflow(plan, e, alt, E: int, C: int):
    """One more stage of No-Token-Left-Behind routing (Appendix B, its figure): every token that has no slot yet is
    offered, in token order, to its next-choice expert `alt[t]` and takes that expert's next free slot if it still
    has one; tokens placed in an earlier stage keep their slots.  Applied to the plan of stage 1 with the second
    choices this is the figure's stage 2; applied again with the third choices it is the iteration the figure's
    caption mentions.  An `alt[t]` of -1 (no expert left to try) leaves the token where it is.  Returns the updated
    plan plus "e_proc", the expert that processes each token (its first choice unless it was rerouted)."""
    e = np.asarray(e, dtype=np.int64)
    alt = np.asarray(alt, dtype=np.int64)
    keep, pos, kept = plan["keep"].copy(), plan["pos"].copy(), plan["kept"].copy()
    e_proc = np.array(plan.get("e_proc", e), dtype=np.int64, copy=True)
    for t in np.flatnonzero(~plan["keep"]):
        i = alt[t]
        if i >= 0 and kept[i] < C:
            pos[t] = kept[i]
            kept[i] += 1
            keep[t] = True
            e_proc[t] = i
    slot = np.where(keep, e_proc * C + pos, -1)
    token_of_slot = np.full(E * C, -1, dtype=np.int64)
    token_of_slot[slot[keep]] = np.flatnonzero(keep)
    out = dict(plan)
    out.update({"pos": pos, "keep": keep, "slot": slot, "token_of_slot": token_of_slot, "kept": kept,
                "e_proc": e_proc, "rerouted": plan.get("rerouted", False) | (keep & ~plan["keep"])})
    return out


def switch_forward(x, W_r, W_in, W_out, capacity_factor: float, alpha: float, router_bias=None,
                   capacity: int | None = None, expert_index=None, experts=None, residual: bool = False,
                   reroute: bool = False, alt_index=None, router_noise=None, router_jitter=None, storage_round=None,
                   geglu: bool = False, expert_keep=None, expert_dropout: float = 0.0, reroute_stages: int = 1):
    """Forward of the Switch FFN layer for one routing group.

    x [T, d]; W_r [d, E]; W_in [E, d, f]; W_out [E, f, d].  `capacity` overrides Eq. 3 when given.
    `expert_index`, when given, replaces the argmax (used to follow a legitimate near-tie flip of the
    device router); the gate is then p[t, expert_index[t]].  `experts`, when given, restricts the
    expert FFN work to that subset (rows of y for other experts' tokens stay 0): the router, plan and
    loss are always computed for every token.  W_in / W_out may be any object indexable by expert.
    `residual` adds the layer's input to its output, y_t = x_t + g_t . E_{e_t}(x_t): the residual connection
    around the Switch FFN layer (Fig. 2), through which a dropped token's representation reaches the next
    layer unchanged (Section 2.2).  "layer_y" always holds the output without it.
    `reroute` adds stage 2 of No-Token-Left-Behind routing (Appendix B): overflowed tokens go to their second-choice
    expert where it has room, and their gate is that expert's probability (Eq. 2 with the expert that processes the
    token); f in the auxiliary loss still counts the argmax (Eq. 5).  `reroute_stages` > 1 iterates (the figure's
    caption: the process can be repeated until virtually no token is dropped): stage 3 offers the tokens that are
    still without a slot to their third choice, and so on.  `alt_index`, when given, replaces the choices (to follow
    a legitimate near-tie flip of the device): [T] for one stage, [stages, T] otherwise.
    `router_jitter` [T, d], when given, multiplies the router's input element by element (input jitter as the text
    describes it, Appendix C): the router sees x . u, the experts see x.  It is an
    input (the caller draws it).  `storage_round`, when given, is applied to x . u: the router's input is a tensor
    of the layer's activation type, so the product is rounded to that type before the router's float32 arithmetic.
    `geglu` replaces the expert's ReLU FFN by the GEGLU FFN of the paper's Table 9 (two expansion matrices whose
    outputs are combined non-linearly): W_in[i] is [d, 2 f] = [W_0 | W_1],
    a = x W_0, b = x W_1, hidden = GELU(a) . b, output = hidden W_out.  "u" then holds the rows [a | b].
    `expert_keep` [E * C, f] (booleans, indexed by slot row) with `expert_dropout` = rate applies expert dropout
    (Section 2.4 / fine-tuning regularisation table: a larger dropout rate on the hidden activations inside every
    expert): the hidden activations are multiplied by keep / (1 - rate), the usual inverted dropout; the
    mask is an input (the caller draws it).
    Returns a dict with every intermediate the staged comparisons need.
    """
    x64 = np.asarray(x, dtype=F64)
    T, d = x64.shape
    E = np.asarray(W_r).shape[1]
    x_router = x64
    if router_jitter is not None:
        x_router = x64 * np.asarray(router_jitter, dtype=F64)
        if storage_round is not None:
            x_router = np.asarray(storage_round(x_router), dtype=F64)
    h = router_logits(x_router, W_r, router_bias, router_noise)
    p = router_probs(h)
    if expert_index is None:
        e, g = top1(p)
    else:
        e = np.asarray(expert_index, dtype=np.int64)
        g = p[np.arange(T), e]
    aux, f, P = load_balance_loss(p, e, alpha)
    C = expert_capacity(T, E, capacity_factor) if capacity is None else int(capacity)
    plan = dispatch_plan(e, E, C)
    e_proc = e
    if reroute:
        given = None if alt_index is None else np.asarray(alt_index, dtype=np.int64).reshape(reroute_stages, T)
        alts, prev = [], e
        for s in range(reroute_stages):
            alt = next_choice(p, prev) if given is None else given[s]
            plan = reroute_overflow(plan, e, alt, E, C)
            alts.append(alt)
            prev = alt
        e_proc = plan["e_proc"]
        g = p[np.arange(T), e_proc]
        plan["alt"] = alts[0] if reroute_stages == 1 else np.stack(alts)
    keep = plan["keep"]

    y = np.zeros((T, d), dtype=F64)
    u = {}                                   # per expert: pre-activation of its kept tokens
    o = np.zeros((T, d), dtype=F64)          # un-gated expert output E_i(x_t); 0 for dropped tokens
    todo = range(E) if experts is None else experts
    for i in todo:
        tok = plan["token_of_slot"][i * C:i * C + int(plan["kept"][i])]   # kept tokens of expert i, in slot order
        if tok.size == 0:
            continue
        u_i = x64[tok] @ np.asarray(W_in[i], dtype=F64)          # h = x W_in  (GEGLU: [a | b] = x [W_0 | W_1])
        if geglu:
            fh = u_i.shape[1] // 2
            a_i = gelu(u_i[:, :fh]) * u_i[:, fh:]                # GELU(x W_0) . (x W_1)
        else:
            a_i = np.maximum(u_i, 0.0)                           # ReLU(h)
        if expert_keep is not None:                              # expert dropout on the hidden activations
            a_i = a_i * (np.asarray(expert_keep)[i * C:i * C + tok.size] / (1.0 - expert_dropout))
        o_i = a_i @ np.asarray(W_out[i], dtype=F64)              # y = ReLU(h) W_out
        u[i] = u_i
        o[tok] = o_i
        y[tok] = g[tok, None] * o_i                              # Eq. 2 with one selected expert
    out = {"h": h, "p": p, "e": e, "g": g, "aux": aux, "f": f, "P": P, "C": C, "layer_y": y,
           "y": x64 + y if residual else y, "o": o, "u": u, "T": T, "E": E, "alpha": alpha, "residual": bool(residual),
           "e_proc": e_proc, "x_router": x_router, "geglu": bool(geglu),
           "expert_keep": None if expert_keep is None else np.asarray(expert_keep, dtype=F64) / (1.0 - expert_dropout),
           "router_jitter": None if router_jitter is None else np.asarray(router_jitter, dtype=F64)}
    out.update(plan)
    return out


def switch_backward(fwd, x, W_r, W_in, W_out, dy, d_aux: float = 1.0, experts=None, want_weight_grads=True):
    """Backward of switch_forward for upstream gradients dy [T, d] (of y) and d_aux (of the auxiliary loss).

    Returns dx [T, d], dW_r [d, E], db [E] (router-bias gradient), dW_in / dW_out as dicts expert -> array
    (experts with no kept token get zeros), plus dgate [T] and dh [T, E] for staged comparisons.
    """
    x64 = np.asarray(x, dtype=F64)
    dy64 = np.asarray(dy, dtype=F64)
    W_r64 = np.asarray(W_r, dtype=F64)
    T, d = x64.shape
    E = W_r64.shape[1]
    p, e, g, keep, alpha = fwd["p"], fwd["e"], fwd["g"], fwd["keep"], fwd["alpha"]

    dx = np.zeros((T, d), dtype=F64)
    dgate = np.zeros(T, dtype=F64)
    dW_in, dW_out = {}, {}
    todo = range(E) if experts is None else experts
    C = fwd["C"]
    e_proc = fwd["e_proc"]
    for i in todo:
        tok = fwd["token_of_slot"][i * C:i * C + int(fwd["kept"][i])]      # the expert's tokens in slot order
        W_in_i = np.asarray(W_in[i], dtype=F64)
        W_out_i = np.asarray(W_out[i], dtype=F64)
        if tok.size == 0:
            if want_weight_grads:
                dW_in[i] = np.zeros_like(W_in_i)
                dW_out[i] = np.zeros_like(W_out_i)
            continue
        u_i = fwd["u"][i]
        do_i = g[tok, None] * dy64[tok]                 # y = g . o        =>  do = g . dy
        dgate[tok] = np.sum(dy64[tok] * fwd["o"][tok], axis=1)   #          =>  dg = <dy, o>
        da_i = do_i @ W_out_i.T                         # o = a W_out
        keep_i = None
        if fwd.get("expert_keep") is not None:          # a = dropout(act(u)): the same factors on the way back
            keep_i = fwd["expert_keep"][i * C:i * C + tok.size]
            da_i = da_i * keep_i
        if fwd.get("geglu", False):
            fh = u_i.shape[1] // 2
            ua, ub = u_i[:, :fh], u_i[:, fh:]
            a_i = gelu(ua) * ub                         # hidden = GELU(a) . b
            du_i = np.concatenate([da_i * ub * gelu_prime(ua), da_i * gelu(ua)], axis=1)
        else:
            a_i = np.maximum(u_i, 0.0)
            du_i = da_i * (u_i > 0.0)                   # a = ReLU(u), ReLU'(0) = 0
        if keep_i is not None:
            a_i = a_i * keep_i                          # the hidden activations that entered W_out
        dx[tok] = du_i @ W_in_i.T                       # u = x W_in
        if want_weight_grads:
            dW_out[i] = a_i.T @ do_i
            dW_in[i] = x64[tok].T @ du_i

    # Router: total loss depends on p through the kept tokens' gates and through P in the auxiliary loss
    # (f is piecewise constant, hence no gradient).  aux = alpha . E . sum_i f_i . (1/T) sum_t p[t, i].
    G = np.broadcast_to((d_aux * alpha * E / T) * fwd["f"][None, :], (T, E)).copy()
    kept_tok = np.flatnonzero(keep)
    G[kept_tok, e_proc[kept_tok]] += dgate[kept_tok]        # the gate is the probability of the expert that processes the token
    dh = p * (G - np.sum(p * G, axis=1, keepdims=True))     # softmax Jacobian applied to G
    dW_r = fwd.get("x_router", x64).T @ dh                 # the router's input (x, or x . u under input jitter)
    db = dh.sum(axis=0)
    dx_router = dh @ W_r64.T
    if fwd.get("router_jitter") is not None:
        dx_router = dx_router * fwd["router_jitter"]        # d(x . u)/dx = u; the storage rounding is passed straight through
    dx = dx + dx_router
    if fwd.get("residual", False):
        dx = dx + dy64                                   # y = x + layer(x): the skip path carries dy to x unchanged
    return {"dx": dx, "dW_r": dW_r, "db": db, "dW_in": dW_in, "dW_out": dW_out, "dgate": dgate, "dh": dh,
            "dx_router": dx_router, "G": G}


def router_backward_given_dgate(p, e, keep, count, dgate, x, W_r, alpha: float, d_aux: float = 1.0):
    """The router's part of the backward pass alone, for a caller-supplied gate gradient dgate [T]."""
    p = np.asarray(p, dtype=F64)
    T, E = p.shape
    f = np.asarray(count, dtype=F64) / T
    G = np.broadcast_to((d_aux * alpha * E / T) * f[None, :], (T, E)).copy()
    kept_tok = np.flatnonzero(keep)
    G[kept_tok, np.asarray(e)[kept_tok]] += np.asarray(dgate, dtype=F64)[kept_tok]
    dh = p * (G - np.sum(p * G, axis=1, keepdims=True))
    x64 = np.asarray(x, dtype=F64)
    return {"dh": dh, "dW_r": x64.T @ dh, "dx_router": dh @ np.asarray(W_r, dtype=F64).T}


# ------------------------------------------------------------------------------------------------------------
# Several routing groups in one call.  The appendix pseudo-code carries a leading [num_cores] dimension on every
# router tensor: each core routes its own tokens_per_core tokens (own capacity from Eq. 3, own f and P in Eq. 5-6),
# the experts are shared, and the loss is the mean over cores and experts times num_experts^2, i.e. the mean of the
# groups' losses.  Here a group is T / G consecutive rows of x.
def switch_forward_groups(x, W_r, W_in, W_out, capacity_factor: float, alpha: float, groups: int, router_bias=None,
                          expert_index=None, experts=None, residual: bool = False, router_noise=None,
                          router_jitter=None, storage_round=None, geglu: bool = False):
    """Forward for G routing groups: switch_forward on each group, results concatenated in token order.

    The merged plan numbers an expert's rows group by group (group 0's kept tokens in token order, then group 1's,
    ...): slot[t] = e_t * (G * C) + (kept tokens of expert e_t in earlier groups) + pos_t, with pos_t and the
    capacity cut taken inside the token's own group.  "aux" is the mean of the groups' losses.
    """
    x64 = np.asarray(x, dtype=F64)
    T = x64.shape[0]
    G = int(groups)
    assert G >= 1 and T % G == 0
    Tg = T // G
    E = np.asarray(W_r).shape[1]
    parts = []
    for g in range(G):
        rows = slice(g * Tg, (g + 1) * Tg)
        ei = None if expert_index is None else np.asarray(expert_index)[rows]
        noise = None if router_noise is None else np.asarray(router_noise)[rows]
        jitter = None if router_jitter is None else np.asarray(router_jitter)[rows]
        parts.append(switch_forward(x64[rows], W_r, W_in, W_out, capacity_factor, alpha, router_bias=router_bias,
                                    expert_index=ei, experts=experts, residual=residual, router_noise=noise,
                                    router_jitter=jitter, storage_round=storage_round, geglu=geglu))
    C = parts[0]["C"]
    cat = lambda k: np.concatenate([q[k] for q in parts], axis=0)
    kept_g = np.stack([q["kept"] for q in parts])                       # [G, E]
    count_g = np.stack([q["count"] for q in parts])
    base_g = np.cumsum(kept_g, axis=0) - kept_g                        # kept tokens of the expert in earlier groups
    e, pos, keep = cat("e"), cat("pos"), cat("keep")
    grp = np.repeat(np.arange(G), Tg)
    slot = np.where(keep, e * (G * C) + base_g[grp, e] + pos, -1)
    token_of_slot = np.full(E * G * C, -1, dtype=np.int64)
    token_of_slot[slot[keep]] = np.flatnonzero(keep)
    out = {"parts": parts, "G": G, "Tg": Tg, "C": C, "E": E, "T": T, "alpha": alpha, "residual": bool(residual),
           "geglu": bool(geglu),
           "aux": float(np.mean([q["aux"] for q in parts])),
           "y": cat("y"), "layer_y": cat("layer_y"), "o": cat("o"), "p": cat("p"), "h": cat("h"), "g": cat("g"),
           "e": e, "pos": pos, "keep": keep, "slot": slot, "token_of_slot": token_of_slot,
           "count": count_g.sum(axis=0), "kept": kept_g.sum(axis=0), "count_g": count_g, "kept_g": kept_g}
    return out


def switch_backward_groups(fwd, x, W_r, W_in, W_out, dy, d_aux: float = 1.0, experts=None, want_weight_grads=True):
    """Backward of switch_forward_groups: each group's backward with d_aux / G (the loss is the groups' mean);
    dx, dgate and dh are concatenated, the weight gradients are summed over the groups."""
    x64 = np.asarray(x, dtype=F64)
    dy64 = np.asarray(dy, dtype=F64)
    G, Tg = fwd["G"], fwd["Tg"]
    outs = []
    for g in range(G):
        rows = slice(g * Tg, (g + 1) * Tg)
        outs.append(switch_backward(fwd["parts"][g], x64[rows], W_r, W_in, W_out, dy64[rows], d_aux=d_aux / G,
                                    experts=experts, want_weight_grads=want_weight_grads))
    cat = lambda k: np.concatenate([q[k] for q in outs], axis=0)
    res = {"dx": cat("dx"), "dgate": cat("dgate"), "dh": cat("dh"), "dx_router": cat("dx_router"),
           "dW_r": sum(q["dW_r"] for q in outs), "db": sum(q["db"] for q in outs), "dW_in": {}, "dW_out": {}}
    if want_weight_grads:
        for i in outs[0]["dW_in"]:
            res["dW_in"][i] = sum(q["dW_in"][i] for q in outs)
            res["dW_out"][i] = sum(q["dW_out"][i] for q in outs)
    return res


# ------------------------------------------------------------------------------------------------------------
# Top-2 routing: the Mixture-of-Experts layer the paper compares with (Eq. 1-2 with the two highest-probability
# experts; "MoE Transformers using top-2 routing" in its comparison tables).  Readings, where the paper gives none:
# the combine weights are the softmax probabilities of Eq. 1 themselves (Eq. 2, no renormalisation over the two);
# every token's first choice is placed before any second choice (token order inside each round), all against the
# same expert capacity; f in the auxiliary loss counts the first choice (the argmax of Eq. 5).
def top2_forward(x, W_r, W_in, W_out, capacity_factor: float, alpha: float, router_bias=None, first_index=None,
                 second_index=None, experts=None, residual: bool = False):
    """Forward of the top-2 layer.  Assignments are numbered v = t for the first choice of token t and v = T + t for
    its second choice; "slot" [2T], "token_of_slot" [E*C] (holding v) and "keep" [2T] describe the plan in that
    numbering, "e" [2T] the expert and "g" [2T] the combine weight of every assignment.
    `residual` adds the layer's input to its output (the residual connection around the layer, Fig. 2; a token both of
    whose assignments overflowed reaches the next layer through it unchanged, Section 2.2); "layer_y" holds the
    output without it."""
    x64 = np.asarray(x, dtype=F64)
    T, d = x64.shape
    E = np.asarray(W_r).shape[1]
    h = router_logits(x64, W_r, router_bias)
    p = router_probs(h)
    a = top1(p)[0] if first_index is None else np.asarray(first_index, dtype=np.int64)
    b = second_choice(p, a) if second_index is None else np.asarray(second_index, dtype=np.int64)
    aux, f, P = load_balance_loss(p, a, alpha)                  # f: first choices only
    C = expert_capacity(T, E, capacity_factor)
    e = np.concatenate([a, b])
    plan = dispatch_plan(e, E, C)                                # first choices of all tokens, then second choices
    keep = plan["keep"]
    tok_of = np.concatenate([np.arange(T), np.arange(T)])       # the token behind an assignment
    g = p[tok_of, e]
    y = np.zeros((T, d), dtype=F64)
    o = np.zeros((2 * T, d), dtype=F64)                          # un-weighted expert output per assignment
    u = {}
    todo = range(E) if experts is None else experts
    for i in todo:
        v = plan["token_of_slot"][i * C:i * C + int(plan["kept"][i])]   # the expert's assignments in slot order
        if v.size == 0:
            continue
        u_i = x64[tok_of[v]] @ np.asarray(W_in[i], dtype=F64)
        o_i = np.maximum(u_i, 0.0) @ np.asarray(W_out[i], dtype=F64)
        u[i] = u_i
        o[v] = o_i
        np.add.at(y, tok_of[v], g[v, None] * o_i)                # Eq. 2: sum over the selected experts
    out = {"h": h, "p": p, "e": e, "g": g, "aux": aux, "f": f, "P": P, "C": C, "layer_y": y,
           "y": x64 + y if residual else y, "residual": bool(residual), "o": o, "u": u, "T": T, "E": E,
           "alpha": alpha, "tok_of": tok_of, "first": a, "second": b}
    out.update(plan)
    out["count_first"] = np.bincount(a, minlength=E)
    return out


def top2_backward(fwd, x, W_r, W_in, W_out, dy, d_aux: float = 1.0, experts=None, want_weight_grads=True):
    """Backward of top2_forward: both kept assignments of a token send gradient to x, to their expert's weights and,
    through their combine weight p[t, e], to the router; f has no gradient."""
    x64 = np.asarray(x, dtype=F64)
    dy64 = np.asarray(dy, dtype=F64)
    W_r64 = np.asarray(W_r, dtype=F64)
    T, d = x64.shape
    E, C = fwd["E"], fwd["C"]
    p, e, g, keep, tok_of, alpha = fwd["p"], fwd["e"], fwd["g"], fwd["keep"], fwd["tok_of"], fwd["alpha"]
    dx = np.zeros((T, d), dtype=F64)
    dgate = np.zeros(2 * T, dtype=F64)
    dW_in, dW_out = {}, {}
    todo = range(E) if experts is None else experts
    for i in todo:
        v = fwd["token_of_slot"][i * C:i * C + int(fwd["kept"][i])]
        W_in_i = np.asarray(W_in[i], dtype=F64)
        W_out_i = np.asarray(W_out[i], dtype=F64)
        if v.size == 0:
            if want_weight_grads:
                dW_in[i] = np.zeros_like(W_in_i)
                dW_out[i] = np.zeros_like(W_out_i)
            continue
        t = tok_of[v]
        u_i = fwd["u"][i]
        a_i = np.maximum(u_i, 0.0)
        do_i = g[v, None] * dy64[t]
        dgate[v] = np.sum(dy64[t] * fwd["o"][v], axis=1)
        du_i = (do_i @ W_out_i.T) * (u_i > 0.0)
        np.add.at(dx, t, du_i @ W_in_i.T)
        if want_weight_grads:
            dW_out[i] = a_i.T @ do_i
            dW_in[i] = x64[t].T @ du_i
    G = np.broadcast_to((d_aux * alpha * E / T) * fwd["f"][None, :], (T, E)).copy()
    kept_v = np.flatnonzero(keep)
    np.add.at(G, (tok_of[kept_v], e[kept_v]), dgate[kept_v])
    dh = p * (G - np.sum(p * G, axis=1, keepdims=True))
    dx_router = dh @ W_r64.T
    dx = dx + dx_router
    if fwd.get("residual", False):
        dx = dx + dy64                                   # y = x + layer(x): the skip path carries dy to x unchanged
    return {"dx": dx, "dW_r": x64.T @ dh, "db": dh.sum(axis=0), "dW_in": dW_in, "dW_out": dW_out,
            "dgate": dgate, "dh": dh, "dx_router": dx_router}
