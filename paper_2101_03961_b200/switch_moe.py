"""ctypes binding of libswitch_moe.so: the same entry points as include/switch_moe.h, taking torch tensors.

Argument marshalling only: every step of the layer runs in the library's CUDA kernels.  PyTorch is used for
device memory and streams.  There is no fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libswitch_moe.so")

BF16, F32 = 0, 1
STAGE_EVENTS = 13
STAGE_NAMES = ["router_fwd", "dispatch_plan", "gather_x", "gemm1_relu", "gemm2_combine", None,
               "gather_dy", "dgrad2_mask", "wgrad2", "dgrad1_scatter", "wgrad1", "router_bwd"]
GEMM_DEFAULT, GEMM_SIMT, GEMM_TC_1CTA = 0, 1, 2

OK = 0
INVALID_ARGUMENT, UNSUPPORTED_SHAPE, WORKSPACE_TOO_SMALL, CUDA_ERROR, DEVICE_TIMEOUT = -1, -2, -3, -4, -5

WS_STATUS, WS_EXPERT_INDEX, WS_GATE, WS_SLOT, WS_TOKEN_OF_SLOT, WS_COUNT, WS_KEPT, WS_PSUM, WS_PROBS, WS_XD, WS_H, \
    WS_DYD, WS_DH, WS_DGATE, WS_DLOGITS, WS_LAYER_Y, WS_EXPERT_PROC, WS_SECOND_CHOICE = range(18)
FLAG_RESIDUAL, FLAG_REROUTE, FLAG_INPUT_JITTER, FLAG_GEGLU, FLAG_TOP2, FLAG_EXPERT_DROPOUT = 1, 2, 4, 8, 16, 32

EXPORTED_SYMBOLS = [
    "switch_moe_capacity", "switch_moe_workspace_bytes", "switch_moe_workspace_view", "switch_moe_fwd",
    "switch_moe_bwd", "switch_moe_router_fwd", "switch_moe_dispatch_plan", "switch_moe_router_bwd",
    "switch_moe_dispatch_plan_static", "switch_moe_step_host", "switch_moe_step_host_enqueue",
    "switch_moe_check_device_status", "switch_moe_launches_per_step", "switch_moe_stage_launches",
    "switch_moe_status_string",
]


class SwitchMoeConfig(ctypes.Structure):
    """Mirror of `switch_moe_config`."""

    _fields_ = [
        ("T", ctypes.c_int32), ("d_model", ctypes.c_int32), ("d_ff", ctypes.c_int32), ("E", ctypes.c_int32),
        ("capacity_factor", ctypes.c_float), ("alpha", ctypes.c_float),
        ("capacity_override", ctypes.c_int32), ("dtype", ctypes.c_int32), ("gemm_path", ctypes.c_int32),
        ("flags", ctypes.c_int32), ("groups", ctypes.c_int32), ("reroute_stages", ctypes.c_int32),
        ("reserved", ctypes.c_int32 * 2),
        ("stage_events", ctypes.POINTER(ctypes.c_void_p)),
        ("router_noise", ctypes.c_void_p),
        ("router_jitter", ctypes.c_void_p),
        ("expert_keep", ctypes.c_void_p),
        ("expert_dropout", ctypes.c_float),
    ]


class SwitchMoeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads libswitch_moe.so (built in-tree by paper_2101_03961_b200.build); raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    path = os.environ.get("SWITCH_MOE_LIBRARY", LIB_PATH)      # override: another build of the same library
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} not found: build it with `python -m paper_2101_03961_b200.build` (there is no fallback path)")
    lib = ctypes.CDLL(path)
    vp, cp = ctypes.c_void_p, ctypes.POINTER(SwitchMoeConfig)
    i32p, szp = ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_size_t)
    lib.switch_moe_capacity.argtypes = [cp, i32p]
    lib.switch_moe_workspace_bytes.argtypes = [cp, szp]
    lib.switch_moe_workspace_view.argtypes = [cp, vp, ctypes.c_int32, ctypes.POINTER(vp), szp]
    lib.switch_moe_fwd.argtypes = [cp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.switch_moe_bwd.argtypes = [cp, vp, ctypes.c_float, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp, vp, vp, vp, vp]
    lib.switch_moe_router_fwd.argtypes = [cp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.switch_moe_dispatch_plan.argtypes = [cp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.switch_moe_dispatch_plan_static.argtypes = [cp, vp, vp, vp, vp, vp, vp]
    lib.switch_moe_router_bwd.argtypes = [cp, vp, vp, vp, ctypes.c_float, vp, ctypes.c_size_t, vp, vp, vp]
    lib.switch_moe_step_host.argtypes = [cp, vp, vp, ctypes.c_float] + [vp] * 15 + [vp, ctypes.c_size_t, vp, vp, vp]
    lib.switch_moe_step_host_enqueue.argtypes = lib.switch_moe_step_host.argtypes + [vp, vp]
    lib.switch_moe_check_device_status.argtypes = [cp, vp, i32p, vp]
    lib.switch_moe_launches_per_step.argtypes = [cp, i32p]
    lib.switch_moe_stage_launches.argtypes = [cp, i32p]
    lib.switch_moe_status_string.argtypes = [ctypes.c_int]
    lib.switch_moe_status_string.restype = ctypes.c_char_p
    for name in EXPORTED_SYMBOLS:
        if name != "switch_moe_status_string":
            getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def make_config(T, d_model, d_ff, E, capacity_factor, alpha=0.01, dtype=BF16, capacity_override=0,
                gemm_path=GEMM_DEFAULT, residual=False, groups=1, reroute=False, input_jitter=False, geglu=False, top2=False, expert_dropout=None, reroute_stages=1) -> SwitchMoeConfig:
    cfg = SwitchMoeConfig()
    cfg.T, cfg.d_model, cfg.d_ff, cfg.E = int(T), int(d_model), int(d_ff), int(E)
    cfg.capacity_factor, cfg.alpha = float(capacity_factor), float(alpha)
    cfg.capacity_override, cfg.dtype, cfg.gemm_path = int(capacity_override), int(dtype), int(gemm_path)
    cfg.flags = ((FLAG_RESIDUAL if residual else 0) | (FLAG_REROUTE if reroute else 0)
                 | (FLAG_INPUT_JITTER if input_jitter else 0) | (FLAG_GEGLU if geglu else 0)
                 | (FLAG_TOP2 if top2 else 0) | (FLAG_EXPERT_DROPOUT if expert_dropout is not None else 0))
    cfg.expert_dropout = float(expert_dropout or 0.0)              # set cfg.expert_keep to the device pointer of the mask     # set cfg.router_jitter to the device pointer of u
    cfg.groups = int(groups)
    cfg.reroute_stages = int(reroute_stages) if reroute else 0
    return cfg


def set_stage_events(cfg: SwitchMoeConfig, events) -> None:
    """Attach STAGE_EVENTS recorded-once torch.cuda.Event objects (enable_timing=True) for per-stage timing, or None."""
    if events is None:
        cfg.stage_events = None
        cfg._stage_event_handles = None
        return
    assert len(events) == STAGE_EVENTS
    handles = (ctypes.c_void_p * STAGE_EVENTS)(*[ev.cuda_event for ev in events])
    cfg._stage_event_handles = handles                      # keep the array alive as long as the config
    cfg.stage_events = ctypes.cast(handles, ctypes.POINTER(ctypes.c_void_p))


def status_string(status: int) -> str:
    return load_library().switch_moe_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise SwitchMoeError(status, where)


def _ptr(t) -> int | None:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int | None:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def switch_moe_capacity(cfg: SwitchMoeConfig) -> int:
    out = ctypes.c_int32(0)
    _check(load_library().switch_moe_capacity(ctypes.byref(cfg), ctypes.byref(out)), "switch_moe_capacity")
    return out.value


def switch_moe_workspace_bytes(cfg: SwitchMoeConfig) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().switch_moe_workspace_bytes(ctypes.byref(cfg), ctypes.byref(out)),
           "switch_moe_workspace_bytes")
    return out.value


def allocate_workspace(cfg: SwitchMoeConfig, device="cuda") -> torch.Tensor:
    """A 1024-byte aligned uint8 device tensor of switch_moe_workspace_bytes(cfg) bytes (torch owns the memory)."""
    n = switch_moe_workspace_bytes(cfg)
    raw = torch.empty(n + 1024, dtype=torch.uint8, device=device)
    off = (-raw.data_ptr()) % 1024
    return raw[off:off + n]


_REGION_DTYPES = {
    WS_STATUS: torch.int32, WS_EXPERT_INDEX: torch.int32, WS_GATE: torch.float32, WS_SLOT: torch.int32,
    WS_TOKEN_OF_SLOT: torch.int32, WS_COUNT: torch.int32, WS_KEPT: torch.int32, WS_PSUM: torch.float32,
    WS_PROBS: torch.float32, WS_DGATE: torch.float32, WS_DLOGITS: torch.float32, WS_EXPERT_PROC: torch.int32,
    WS_SECOND_CHOICE: torch.int32,
}


def switch_moe_workspace_view(cfg: SwitchMoeConfig, workspace: torch.Tensor, region: int) -> torch.Tensor:
    """A typed 1-D tensor aliasing one region of the workspace (no copy)."""
    ptr, nbytes = ctypes.c_void_p(0), ctypes.c_size_t(0)
    _check(load_library().switch_moe_workspace_view(ctypes.byref(cfg), workspace.data_ptr(), int(region),
                                                    ctypes.byref(ptr), ctypes.byref(nbytes)),
           "switch_moe_workspace_view")
    off = ptr.value - workspace.data_ptr()
    raw = workspace[off:off + nbytes.value]
    dt = _REGION_DTYPES.get(region, torch.bfloat16 if cfg.dtype == BF16 else torch.float32)
    return raw.view(dt)


def switch_moe_fwd(cfg, x, W_r, router_bias, W_in, W_out, y, aux_loss, workspace, stream=None) -> None:
    _check(load_library().switch_moe_fwd(ctypes.byref(cfg), _ptr(x), _ptr(W_r), _ptr(router_bias), _ptr(W_in),
                                         _ptr(W_out), _ptr(y), _ptr(aux_loss), _ptr(workspace), workspace.numel(),
                                         _stream(stream)), "switch_moe_fwd")


def switch_moe_bwd(cfg, dy, d_aux, x, W_r, W_in, W_out, y, workspace, dx, dW_r, dW_in, dW_out, stream=None) -> None:
    _check(load_library().switch_moe_bwd(ctypes.byref(cfg), _ptr(dy), float(d_aux), _ptr(x), _ptr(W_r), _ptr(W_in),
                                         _ptr(W_out), _ptr(y), _ptr(workspace), workspace.numel(), _ptr(dx),
                                         _ptr(dW_r), _ptr(dW_in), _ptr(dW_out), _stream(stream)), "switch_moe_bwd")


def switch_moe_router_fwd(cfg, x, W_r, router_bias, workspace, stream=None) -> None:
    _check(load_library().switch_moe_router_fwd(ctypes.byref(cfg), _ptr(x), _ptr(W_r), _ptr(router_bias),
                                                _ptr(workspace), workspace.numel(), _stream(stream)),
           "switch_moe_router_fwd")


def switch_moe_dispatch_plan(cfg, expert_index, aux_loss, workspace, stream=None) -> None:
    _check(load_library().switch_moe_dispatch_plan(ctypes.byref(cfg), _ptr(expert_index), _ptr(aux_loss),
                                                   _ptr(workspace), workspace.numel(), _stream(stream)),
           "switch_moe_dispatch_plan")


def switch_moe_dispatch_plan_static(cfg, expert_index, count, kept, slot, token_of_slot, stream=None) -> None:
    """Dispatch plan without a workspace and without any allocation (scratch is a static array inside the library);
    for callers that cannot call cudaMalloc.  Outputs go to the four caller-owned int32 tensors."""
    _check(load_library().switch_moe_dispatch_plan_static(ctypes.byref(cfg), _ptr(expert_index), _ptr(count),
                                                          _ptr(kept), _ptr(slot), _ptr(token_of_slot),
                                                          _stream(stream)), "switch_moe_dispatch_plan_static")


def switch_moe_router_bwd(cfg, x, W_r, dgate, d_aux, workspace, dx_router, dW_r, stream=None) -> None:
    _check(load_library().switch_moe_router_bwd(ctypes.byref(cfg), _ptr(x), _ptr(W_r), _ptr(dgate), float(d_aux),
                                                _ptr(workspace), workspace.numel(), _ptr(dx_router), _ptr(dW_r),
                                                _stream(stream)), "switch_moe_router_bwd")


def switch_moe_step_host(cfg, x_host, dy_host, d_aux, W_r, router_bias, W_in, W_out, x_dev, dy_dev, y_dev, dx_dev,
                         aux_dev, dW_r, dW_in, dW_out, y_host, dx_host, aux_host, workspace, stream=None,
                         h2d_stream=None, d2h_stream=None) -> None:
    _check(load_library().switch_moe_step_host(
        ctypes.byref(cfg), _ptr(x_host), _ptr(dy_host), float(d_aux), _ptr(W_r), _ptr(router_bias), _ptr(W_in),
        _ptr(W_out), _ptr(x_dev), _ptr(dy_dev), _ptr(y_dev), _ptr(dx_dev), _ptr(aux_dev), _ptr(dW_r), _ptr(dW_in),
        _ptr(dW_out), _ptr(y_host), _ptr(dx_host), _ptr(aux_host), _ptr(workspace), workspace.numel(),
        _stream(stream), None if h2d_stream is None else _stream(h2d_stream),
        None if d2h_stream is None else _stream(d2h_stream)), "switch_moe_step_host")


def switch_moe_step_host_enqueue(cfg, x_host, dy_host, d_aux, W_r, router_bias, W_in, W_out, x_dev, dy_dev, y_dev, dx_dev,
                                 aux_dev, dW_r, dW_in, dW_out, y_host, dx_host, aux_host, workspace, stream, h2d_stream,
                                 d2h_stream, slot_free_event, step_done_event) -> None:
    """Non-blocking step: `slot_free_event` / `step_done_event` are torch.cuda.Event objects (the first may be None).
    torch creates the CUDA event behind an Event object on its first record(), so `step_done_event` is recorded once
    on `d2h_stream` here before its handle is passed down (the library records it again after the last download)."""
    if not step_done_event.cuda_event:
        step_done_event.record(d2h_stream)
    _check(load_library().switch_moe_step_host_enqueue(
        ctypes.byref(cfg), _ptr(x_host), _ptr(dy_host), float(d_aux), _ptr(W_r), _ptr(router_bias), _ptr(W_in),
        _ptr(W_out), _ptr(x_dev), _ptr(dy_dev), _ptr(y_dev), _ptr(dx_dev), _ptr(aux_dev), _ptr(dW_r), _ptr(dW_in),
        _ptr(dW_out), _ptr(y_host), _ptr(dx_host), _ptr(aux_host), _ptr(workspace), workspace.numel(),
        _stream(stream), _stream(h2d_stream), _stream(d2h_stream),
        None if slot_free_event is None else ctypes.c_void_p(slot_free_event.cuda_event),
        ctypes.c_void_p(step_done_event.cuda_event)), "switch_moe_step_host_enqueue")


def switch_moe_check_device_status(cfg, workspace, stream=None) -> list:
    """Synchronises the stream; raises SwitchMoeError on a device-side timeout, returns the raw status words."""
    info = (ctypes.c_int32 * 16)()
    rc = load_library().switch_moe_check_device_status(ctypes.byref(cfg), _ptr(workspace), info, _stream(stream))
    if rc != OK:
        raise SwitchMoeError(rc, f"switch_moe_check_device_status info={list(info)}")
    return list(info)


def switch_moe_launches_per_step(cfg) -> int:
    out = ctypes.c_int32(0)
    _check(load_library().switch_moe_launches_per_step(ctypes.byref(cfg), ctypes.byref(out)),
           "switch_moe_launches_per_step")
    return out.value


def switch_moe_stage_launches(cfg) -> dict:
    """Kernel launches per stage, keyed by STAGE_NAMES."""
    out = (ctypes.c_int32 * (STAGE_EVENTS - 1))()
    _check(load_library().switch_moe_stage_launches(ctypes.byref(cfg), out), "switch_moe_stage_launches")
    return {name: int(out[i]) for i, name in enumerate(STAGE_NAMES) if name is not None}
