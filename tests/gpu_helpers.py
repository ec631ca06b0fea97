"""Shared plumbing of the GPU parity tests: upload seeded inputs, run the CUDA library through its C ABI, fetch
results as float64 numpy arrays, and compare with the CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import switch_oracle as so
from paper_2101_03961_b200 import build as sbuild
from paper_2101_03961_b200 import inputs as si
from paper_2101_03961_b200 import switch_moe as sm

# Tolerances.  Every floating-point tensor is held to two bounds with the same number `tol`:
#   the relative Frobenius error        ||a - b||_F <= tol ||b||_F                  (the tensor as a whole), and
#   an element-wise bound               |a_i - b_i| <= 2 tol (rms_i(b) + |b_i|)     (no single element may be off:
#                                                                                    a zeroed row or one wrong value
#                                                                                    disappears in a norm),
# where rms_i(b) is the root mean square of b over the whole tensor, over the element's row or over its column
# (last two axes), whichever is largest: rounding noise scales with the operands that meet in the element, and those
# scale by row (a token's gate multiplies its whole row of y, dY_d and dx) or by column (a hidden unit's activity
# scales its column of dW_in, an expert's gate gradients its column of dW_r), so one global rms would hold the rows
# and columns that carry most of the signal to a tighter bound than their own rounding allows.
# The fp32 router: 1e-5.  bf16 layer outputs and weight gradients: 2e-2 (one bf16 rounding is up to 2^-8 = 4e-3
# relative; H, dY_d, dH and the result are each rounded once and the products accumulate in fp32).  All-fp32
# configuration: 2e-4 (fp32 accumulation over d_ff terms).
# Why the element-wise bound carries a factor ELEM_FACTOR = 2: an element of a product of K terms carries rounding
# noise with a standard deviation of about 2^-9 / sqrt(3) of the local rms per rounded operand in its chain (two to
# four operands: 2e-3 to 4e-3 of the local rms, which is also what the measured Frobenius errors are), and the
# largest of the 10^7 to 2 x 10^8 elements of one tensor lies 5.5 to 6.5 standard deviations out: 1.2e-2 to 2.5e-2
# of the local rms on correct results (measured: up to 2.46e-2, GEGLU experts' dW_out).  A bound at `tol` itself
# would sit inside that tail; at 2 tol it is 10 standard deviations out, and every structural fault (a zeroed or
# stale row, a swapped or missing element) is still 10 to 50 times beyond it.
ELEM_FACTOR = 2.0
TOL_ROUTER = 1e-5
TOL_BF16 = 2e-2
TOL_F32 = 2e-4
FLIP_GAP = 1e-4
RELU_GAP = 1e-4


class Err(float):
    """The larger of the relative Frobenius error and the element-wise measure divided by ELEM_FACTOR, comparable
    with a tolerance like a plain float (value <= tol means both bounds hold); its repr names both measures and the
    worst element so that a failing assert shows where the tensors differ."""

    def __new__(cls, frob, elem, where, got, want):
        self = super().__new__(cls, max(frob, elem / ELEM_FACTOR) if np.isfinite(frob) and np.isfinite(elem)
                               else float("nan"))
        self.frob, self.elem, self.where, self.got, self.want = frob, elem, where, got, want
        return self

    def __repr__(self):
        return (f"{float(self):.3e} (frobenius {self.frob:.3e}; element-wise {self.elem:.3e} at {self.where}: "
                f"got {self.got:.6g}, want {self.want:.6g})")

    __str__ = __repr__


def rel_err(a, b) -> Err:
    """Relative Frobenius error and the element-wise measure max_i |a_i - b_i| / (rms_i(b) + |b_i|) of `a` against
    the oracle's `b` (rms_i: the largest of the rms of the tensor, of the element's row and of its column); the
    returned number is the larger of the first measure and the second divided by ELEM_FACTOR, so that `<= tol` states
    both bounds (NaN if anything is not finite)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    assert a.shape == b.shape, (a.shape, b.shape)
    if a.size == 0:
        return Err(0.0, 0.0, (), 0.0, 0.0)
    diff = np.abs(a - b)
    den = np.linalg.norm(b)
    frob = float(np.linalg.norm(diff) / den) if den > 0 else float(np.linalg.norm(diff))
    rms = np.full_like(b, den / np.sqrt(b.size))
    if b.ndim >= 2:
        sq = b * b
        rms = np.maximum(rms, np.sqrt(sq.mean(axis=-1, keepdims=True)))      # the element's row
        rms = np.maximum(rms, np.sqrt(sq.mean(axis=-2, keepdims=True)))      # the element's column
    ratio = diff / (rms + np.abs(b)) if den > 0 else diff
    flat = int(np.nanargmax(np.where(np.isfinite(ratio), ratio, np.inf)))
    where = tuple(int(v) for v in np.unravel_index(flat, a.shape))
    return Err(frob, float(ratio.reshape(-1)[flat]), where, float(a.reshape(-1)[flat]), float(b.reshape(-1)[flat]))


def to_dev(a: np.ndarray, dtype: int) -> torch.Tensor:
    """float32 numpy -> device tensor in the layer's activation dtype (bf16 bits uploaded as-is)."""
    if dtype == sm.BF16:
        bits = si.to_bf16_bits(a)
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16).reshape(a.shape)
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


class GpuLayer:
    """Device buffers of one layer call plus the library calls on them."""

    def __init__(self, cfg: si.SwitchConfig, data: dict, gemm_path=sm.GEMM_DEFAULT, capacity_override=0,
                 residual=False, groups=1, reroute=False, geglu=False, top2=False, reroute_stages=1):
        sbuild.build()
        keep = data.get("expert_keep")
        geglu = geglu or cfg.geglu
        jit = data.get("router_jitter")
        self.scfg = cfg
        self.cfg = sm.make_config(cfg.T, cfg.d_model, cfg.d_ff, cfg.E, cfg.capacity_factor, cfg.alpha,
                                  dtype=cfg.dtype, capacity_override=capacity_override, gemm_path=gemm_path,
                                  residual=residual, groups=groups, reroute=reroute, input_jitter=jit is not None,
                                  geglu=geglu, top2=top2, reroute_stages=reroute_stages,
                                  expert_dropout=data.get("expert_dropout") if keep is not None else None)
        dt = cfg.dtype
        self.x = to_dev(data["x"], dt)
        self.dy = to_dev(data["dy"], dt)
        self.W_r = torch.from_numpy(np.ascontiguousarray(data["W_r"], dtype=np.float32)).cuda()
        b = data.get("router_bias")
        self.bias = None if b is None else torch.from_numpy(np.ascontiguousarray(b, dtype=np.float32)).cuda()
        n = data.get("router_noise")
        self.noise = None if n is None else torch.from_numpy(np.ascontiguousarray(n, dtype=np.float32)).cuda()
        if self.noise is not None:
            self.cfg.router_noise = self.noise.data_ptr()
        self.jitter = None if jit is None else to_dev(jit, dt)
        if self.jitter is not None:
            self.cfg.router_jitter = self.jitter.data_ptr()
        self.keep = None
        if keep is not None:
            self.keep = torch.from_numpy(si.pack_keep_bits(keep).view(np.int32)).cuda()
            self.cfg.expert_keep = self.keep.data_ptr()
        self.W_in = to_dev(data["W_in"], dt)
        self.W_out = to_dev(data["W_out"], dt)
        tdt = torch.bfloat16 if dt == sm.BF16 else torch.float32
        # outputs start as NaN so that any element the library fails to write shows up
        self.y = torch.full_like(self.x, float("nan"))
        self.dx = torch.full_like(self.x, float("nan"))
        self.dW_in = torch.full_like(self.W_in, float("nan"))
        self.dW_out = torch.full_like(self.W_out, float("nan"))
        self.dW_r = torch.full_like(self.W_r, float("nan"))
        self.aux = torch.full((1,), float("nan"), dtype=torch.float32, device="cuda")
        self.ws = sm.allocate_workspace(self.cfg)
        self.ws.fill_(0xFF)                       # stale workspace contents must never leak into results
        self.C = sm.switch_moe_capacity(self.cfg)
        self.view(sm.WS_STATUS).zero_()
        assert tdt == self.x.dtype

    def view(self, region):
        return sm.switch_moe_workspace_view(self.cfg, self.ws, region)

    def fwd(self):
        sm.switch_moe_fwd(self.cfg, self.x, self.W_r, self.bias, self.W_in, self.W_out, self.y, self.aux, self.ws)
        sm.switch_moe_check_device_status(self.cfg, self.ws)

    def bwd(self, d_aux=1.0):
        sm.switch_moe_bwd(self.cfg, self.dy, d_aux, self.x, self.W_r, self.W_in, self.W_out, self.y, self.ws, self.dx,
                          self.dW_r, self.dW_in, self.dW_out)
        sm.switch_moe_check_device_status(self.cfg, self.ws)

    def expert_index(self) -> np.ndarray:
        return self.view(sm.WS_EXPERT_INDEX).cpu().numpy().astype(np.int64)


def check_flips(gpu_e: np.ndarray, ora: dict) -> int:
    """Argmax flips are legitimate only where the oracle's top-2 probability gap is below FLIP_GAP."""
    diff = np.flatnonzero(gpu_e != ora["e"])
    if diff.size:
        srt = np.sort(ora["p"][diff], axis=1)
        gap = srt[:, -1] - srt[:, -2]
        assert np.all(gap < FLIP_GAP), f"{diff.size} flips, largest gap {gap.max():.3e}"
        # the expert the device picked must be the oracle's runner-up-or-tied maximum
        assert np.all(ora["p"][diff, gpu_e[diff]] >= srt[:, -2] - 1e-12)
    return int(diff.size)


def follow_relu_flips(fwd: dict, hidden_rows, experts=None) -> int:
    """ReLU'(u) = [u > 0] is a discrete decision taken from a floating-point number.  The device takes it from its
    own float32-accumulated pre-activation (the sign it stored with the hidden activation); where that sign differs
    from the oracle's float64 one, a whole term of the backward pass appears or vanishes (one token's contribution to
    a column of dW_in and to its dx row), which is not a rounding error of any size.  As with argmax flips, such a
    flip is legitimate only inside a gap -- |u| <= RELU_GAP . rms(u) of the expert's pre-activations, a few float32
    accumulation errors -- and the oracle's backward pass then follows the device's decision: the oracle's u is
    nudged to +-1e-300 at those elements (the forward values change by less than the gap).
    `hidden_rows(i, k)` returns the device's hidden activations of expert i's first k slot rows as numpy.
    Returns the number of flips.  GEGLU experts have no such decision."""
    if fwd.get("geglu", False):
        return 0
    parts = fwd["parts"] if "parts" in fwd else [fwd]
    todo = sorted({i for q in parts for i in q["u"]}) if experts is None else experts
    flips = 0
    for i in todo:
        k = sum(q["u"][i].shape[0] for q in parts if i in q["u"])
        if k == 0:
            continue
        got = np.asarray(hidden_rows(i, k)) > 0
        row = 0
        for q in parts:                                       # the expert's rows, routing group by routing group
            if i not in q["u"]:
                continue
            u = q["u"][i]
            m = got[row:row + u.shape[0]]
            differ = m != (u > 0.0)
            if fwd.get("expert_keep") is not None:             # a dropped-out unit's sign is not observable (nor used)
                differ &= fwd["expert_keep"][i * fwd["C"] + row:i * fwd["C"] + row + u.shape[0]] > 0
            if differ.any():
                gap = RELU_GAP * np.sqrt(np.mean(u * u))
                assert np.all(np.abs(u[differ]) <= gap), (i, int(differ.sum()), float(np.abs(u[differ]).max()), gap)
                u[differ] = np.where(m[differ], 1e-300, -1e-300)
                flips += int(differ.sum())
            row += u.shape[0]
    return flips


def check_second_choice(gpu_alt: np.ndarray, p: np.ndarray, e: np.ndarray, overflowed: np.ndarray) -> np.ndarray:
    """The device's second choice of every overflowed token must be the oracle's, except where the second and third
    probabilities are closer than FLIP_GAP; tokens that kept their slot carry -1.  Returns the choices to follow."""
    want = so.second_choice(p, e)
    assert np.all(gpu_alt[~overflowed] == -1)
    diff = np.flatnonzero(overflowed & (gpu_alt != want))
    if diff.size:
        assert np.all(gpu_alt[diff] != e[diff]) and np.all(gpu_alt[diff] >= 0)
        gap = p[diff, want[diff]] - p[diff, gpu_alt[diff]]
        assert np.all(np.abs(gap) < FLIP_GAP), f"{diff.size} second-choice flips, largest gap {np.abs(gap).max():.3e}"
    return np.where(overflowed, gpu_alt, want)


def check_next_choices(gpu_alt: np.ndarray, p: np.ndarray, e: np.ndarray, plan: dict, E: int, C: int) -> np.ndarray:
    """The further stages of No-Token-Left-Behind routing, stage by stage.  gpu_alt [stages, T]: the device's next
    choice of every token that had no slot when the stage began must be the expert with the highest probability
    among those the token has not tried yet (lowest index on ties) -- the oracle's next_choice, as long as no
    near-tie has flipped -- except where the two probabilities are closer than FLIP_GAP; tokens that have a slot
    carry -1.  The oracle's plan then follows the device's choices.  Returns the choices to follow, [stages, T]."""
    T = e.shape[0]
    gpu_alt = gpu_alt.reshape(-1, T)
    tried = np.zeros(p.shape, dtype=bool)
    tried[np.arange(T), e] = True
    prev, flipped, follow = e, False, []
    for got in gpu_alt:
        waiting = ~plan["keep"]
        left = np.where(tried, -np.inf, p)
        want = np.where(np.isfinite(left.max(axis=1)), np.argmax(left, axis=1), -1)
        if not flipped:                                       # (a token whose first choice flipped inside the gap has
            same = e == np.argmax(p, axis=1)                  # the oracle's own argmax still untried: its ranking walk
            np.testing.assert_array_equal(want[same], so.next_choice(p, prev)[same])   # starts one place later)
        assert np.all(got[~waiting] == -1)
        diff = np.flatnonzero(waiting & (got != want))
        if diff.size:
            flipped = True
            assert np.all(got[diff] >= 0) and not tried[diff, got[diff]].any()
            gap = p[diff, want[diff]] - p[diff, got[diff]]
            assert np.all(np.abs(gap) < FLIP_GAP), f"{diff.size} next-choice flips, largest gap {np.abs(gap).max():.3e}"
        nxt = np.where(waiting, got, want)
        ok = nxt >= 0
        tried[np.flatnonzero(ok), nxt[ok]] = True
        plan = so.reroute_overflow(plan, e, nxt, E, C)
        follow.append(nxt)
        prev = nxt
    return np.stack(follow)


def oracle_following(cfg: si.SwitchConfig, data: dict, gpu_e: np.ndarray, capacity=None, experts=None,
                     residual=False, groups=1, gpu_alt=None, geglu=False):
    """Oracle forward with the device's expert choice (identical unless a near-tie flipped), after checking flips."""
    jit_kw = {"geglu": True} if (geglu or cfg.geglu) else {}
    if data.get("expert_keep") is not None:
        jit_kw.update({"expert_keep": data["expert_keep"], "expert_dropout": data["expert_dropout"]})
    if data.get("router_jitter") is not None:                  # the router sees x . u rounded to the activation type
        jit_kw.update({"router_jitter": data["router_jitter"], "storage_round": si.storage_round(cfg)})
    if groups > 1:
        assert capacity is None
        first = so.switch_forward_groups(data["x"], data["W_r"], data["W_in"], data["W_out"], cfg.capacity_factor,
                                         cfg.alpha, groups, router_bias=data.get("router_bias"), experts=[],
                                         router_noise=data.get("router_noise"), **jit_kw)
        flips = check_flips(gpu_e, first)
        fwd = so.switch_forward_groups(data["x"], data["W_r"], data["W_in"], data["W_out"], cfg.capacity_factor,
                                       cfg.alpha, groups, router_bias=data.get("router_bias"), expert_index=gpu_e,
                                       experts=experts, residual=residual, router_noise=data.get("router_noise"),
                                       **jit_kw)
        fwd["flips"] = flips
        return fwd
    first = so.switch_forward(data["x"], data["W_r"], data["W_in"], data["W_out"], cfg.capacity_factor, cfg.alpha,
                              router_bias=data.get("router_bias"), capacity=capacity, experts=[],
                              router_noise=data.get("router_noise"), **jit_kw)
    flips = check_flips(gpu_e, first)
    alt = None
    stages = 1
    if gpu_alt is not None:                                   # the further stages of No-Token-Left-Behind routing
        stage1 = so.switch_forward(data["x"], data["W_r"], data["W_in"], data["W_out"], cfg.capacity_factor,
                                   cfg.alpha, router_bias=data.get("router_bias"), capacity=capacity,
                                   expert_index=gpu_e, experts=[], router_noise=data.get("router_noise"), **jit_kw)
        alt = check_next_choices(gpu_alt, stage1["p"], gpu_e, stage1, cfg.E, stage1["C"])
        stages = alt.shape[0]
    fwd = so.switch_forward(data["x"], data["W_r"], data["W_in"], data["W_out"], cfg.capacity_factor, cfg.alpha,
                            router_bias=data.get("router_bias"), capacity=capacity, expert_index=gpu_e,
                            experts=experts, residual=residual, reroute=gpu_alt is not None, alt_index=alt,
                            reroute_stages=stages, router_noise=data.get("router_noise"), **jit_kw)
    fwd["flips"] = flips
    return fwd


def skip_path_ok(got, want_sum, want_layer, tol, dtype, roundings=2) -> bool:
    """Bound for an output that carries the skip path (y = x + layer, dx = dy + layer gradient): the layer term is
    held to `tol` as everywhere else, and the stored sum may be off by the roundings of the storage type it went
    through (y: the term is rounded, then the sum; dx: the expert term, the sum, and the sum again when the router's
    gradient is added).  As a whole: `roundings` x 2^-9 (bfloat16; the rms of a rounding) relative to the sum; element
    by element: `roundings` x 2^-8 (its worst case, for a value just above a power of two) relative to the sum's
    element, plus the layer term's element-wise bound."""
    rnd = 2.0 ** -9 if dtype == sm.BF16 else 2.0 ** -24
    got = np.asarray(got, dtype=np.float64)
    want_layer = np.asarray(want_layer, dtype=np.float64)
    diff = np.abs(got - want_sum)
    whole = np.linalg.norm(diff) <= roundings * rnd * np.linalg.norm(want_sum) + tol * np.linalg.norm(want_layer)
    rms = np.full_like(want_layer, np.linalg.norm(want_layer) / np.sqrt(max(want_layer.size, 1)))
    if want_layer.ndim >= 2:
        rms = np.maximum(rms, np.sqrt((want_layer ** 2).mean(axis=-1, keepdims=True)))
    each = diff <= 2 * roundings * rnd * np.abs(want_sum) + ELEM_FACTOR * tol * (rms + np.abs(want_layer))
    if not (whole and each.all()):
        worst = np.unravel_index(int(np.argmax(diff - 2 * roundings * rnd * np.abs(want_sum)
                                               - ELEM_FACTOR * tol * (rms + np.abs(want_layer)))), diff.shape)
        print("skip_path_ok: whole", bool(whole), "worst element", worst, "got", got[worst], "want", want_sum[worst],
              "layer term", want_layer[worst])
    return bool(whole and each.all())


def expert_preactivation(fwd: dict, i: int):
    """Rows of u = x W_in for expert i in slot order (group by group when the call had several routing groups)."""
    if "parts" not in fwd:
        return fwd["u"].get(i)
    rows = [q["u"][i] for q in fwd["parts"] if i in q["u"]]
    return np.concatenate(rows, axis=0) if rows else None


def expert_hidden(fwd: dict, i: int):
    """The hidden activations of expert i's rows in slot order: ReLU(u), or GELU(a) . b for GEGLU experts."""
    u = expert_preactivation(fwd, i)
    if fwd.get("geglu", False):
        fh = u.shape[1] // 2
        hidden = so.gelu(u[:, :fh]) * u[:, fh:]
    else:
        hidden = np.maximum(u, 0.0)
    if fwd.get("expert_keep") is not None:                       # factors keep / (1 - rate), by slot row
        hidden = hidden * fwd["expert_keep"][i * fwd["C"]:i * fwd["C"] + hidden.shape[0]]
    return hidden
