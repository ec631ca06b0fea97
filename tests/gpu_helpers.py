"""Shared plumbing of the GPU parity tests: upload seeded inputs, run the CUDA library through its C ABI, fetch
results as float64 numpy arrays, and compare with the CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import switch_oracle as so
from paper_2101_03961_b200 import build as sbuild
from paper_2101_03961_b200 import inputs as si
from paper_2101_03961_b200 import switch_moe as sm

# Tolerances (relative Frobenius error per tensor).  The fp32 router: 1e-5.  bf16 layer outputs and weight
# gradients: 2e-2 (one bf16 rounding is 2^-9 = 2e-3 relative; H, dY_d, dH and the result are each rounded once
# and the products accumulate in fp32).  All-fp32 configuration: 2e-4 (fp32 accumulation over d_ff terms).
TOL_ROUTER = 1e-5
TOL_BF16 = 2e-2
TOL_F32 = 2e-4
FLIP_GAP = 1e-4


def rel_err(a, b) -> float:
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))


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
                 residual=False, groups=1, reroute=False, geglu=False, top2=False):
        sbuild.build()
        keep = data.get("expert_keep")
        geglu = geglu or cfg.geglu
        jit = data.get("router_jitter")
        self.scfg = cfg
        self.cfg = sm.make_config(cfg.T, cfg.d_model, cfg.d_ff, cfg.E, cfg.capacity_factor, cfg.alpha,
                                  dtype=cfg.dtype, capacity_override=capacity_override, gemm_path=gemm_path,
                                  residual=residual, groups=groups, reroute=reroute, input_jitter=jit is not None,
                                  geglu=geglu, top2=top2,
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
    if gpu_alt is not None:                                   # stage 2 of No-Token-Left-Behind routing
        stage1 = so.switch_forward(data["x"], data["W_r"], data["W_in"], data["W_out"], cfg.capacity_factor,
                                   cfg.alpha, router_bias=data.get("router_bias"), capacity=capacity,
                                   expert_index=gpu_e, experts=[], router_noise=data.get("router_noise"), **jit_kw)
        alt = check_second_choice(gpu_alt, stage1["p"], gpu_e, ~stage1["keep"])
    fwd = so.switch_forward(data["x"], data["W_r"], data["W_in"], data["W_out"], cfg.capacity_factor, cfg.alpha,
                            router_bias=data.get("router_bias"), capacity=capacity, expert_index=gpu_e,
                            experts=experts, residual=residual, reroute=gpu_alt is not None, alt_index=alt,
                            router_noise=data.get("router_noise"), **jit_kw)
    fwd["flips"] = flips
    return fwd


def skip_path_ok(got, want_sum, want_layer, tol, dtype) -> bool:
    """Bound for an output that carries the skip path (y = x + layer, dx = dy + layer gradient): the layer term is
    held to `tol` as everywhere else, and the stored sum may be off by two roundings of the storage type (the term is
    rounded, then the sum): 2 x 2^-9 for bfloat16, 2 x 2^-24 for float32, relative to the sum."""
    ulp2 = 2.0 ** -8 if dtype == sm.BF16 else 2.0 ** -23
    got = np.asarray(got, dtype=np.float64)
    err = np.linalg.norm(got - want_sum)
    return bool(err <= ulp2 * np.linalg.norm(want_sum) + tol * np.linalg.norm(want_layer))


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
