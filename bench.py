#!/usr/bin/env python
"""Benchmark of the Switch FFN layer (forward + backward) on B200: tokens/s, roofline fraction, CPU-oracle baseline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload switch_base]

One step = one switch_moe_fwd + one switch_moe_bwd over a batch of T synthetic tokens (every hot-path stage).
With N > 1 (launched by torchrun) every rank runs an independent replica on its own GPU: the layer has no
exchange step on one device, so there is no collective on the data path ("replicas only", weak scaling).
`--impl reference` times the CPU oracle on the same workload on the host cores (each step one whole pass).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2101_03961_b200 import inputs as si  # noqa: E402

METRIC = "switch_moe_layer_fwd_bwd_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return json.load(open(path)), "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


def load_captured_traffic(cfg):
    """DRAM bytes per expert product from the committed ncu summary (dram__bytes_read.sum + dram__bytes_write.sum of
    one capture, mean over the six products), scaled to this workload by its number of experts when the capture's
    per-expert shape (d_model, d_ff, tokens per expert) is this workload's: traffic is proportional to E then.
    Returns None when no capture of this shape is recorded."""
    path = os.path.join(ROOT, "profiles", "expert_gemm_dram_traffic.txt")
    if not os.path.exists(path):
        return None
    rec = {}
    for line in open(path):
        if "=" in line and not line.lstrip().startswith("#"):
            k, v = line.split("=", 1)
            rec[k.strip()] = v.strip()
    try:
        same = (int(rec["d_model"]), int(rec["d_ff"])) == (cfg.d_model, cfg.d_ff) and \
            int(rec["T"]) * cfg.E == cfg.T * int(rec["E"]) and rec.get("geglu", "0") == ("1" if cfg.geglu else "0")
        if not same:
            return None
        return {"bytes_per_product": float(rec["dram_bytes_per_product"]) * cfg.E / int(rec["E"]),
                "source": f"ncu capture of {rec.get('workload')} at commit {rec.get('commit')} "
                          f"(profiles/expert_gemm_dram_traffic.txt), scaled by E = {cfg.E}/{rec['E']}"}
    except (KeyError, ValueError):
        return None


def same_run_peaks(device, seconds: float = 2.0):
    """Copy bandwidth and dense bf16 matmul throughput of this box, measured with torch right after the timed regions
    (harness side only: nothing of the layer runs here).  Clocks and power limits differ between boxes of the pool, so
    these sit beside the fractions that are quoted against the generated peaks."""
    import torch
    n = 512 * 1024 * 1024                                     # bf16 elements per buffer: 1 GiB read + 1 GiB written
    a = torch.zeros(n, dtype=torch.bfloat16, device=device)
    b = torch.empty_like(a)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, reps=1):
        torch.cuda.synchronize(device)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize(device)
        return e0.elapsed_time(e1) * 1e-3 / reps

    for _ in range(2):
        b.copy_(a)
    copy_s = min(timed(lambda: b.copy_(a)) for _ in range(10))
    del a, b
    m = 8192
    A = torch.randn(m, m, device=device).to(torch.bfloat16)
    B = torch.randn(m, m, device=device).to(torch.bfloat16)
    C = torch.empty(m, m, dtype=torch.bfloat16, device=device)
    for _ in range(3):
        torch.matmul(A, B, out=C)
    burst_s = min(timed(lambda: torch.matmul(A, B, out=C)) for _ in range(10))
    loops = max(10, int(seconds / burst_s))
    sustained_s = timed(lambda: torch.matmul(A, B, out=C), reps=loops)
    flops = 2.0 * m * m * m
    return {"hbm_gbs": 2 * n * 2 / copy_s / 1e9, "bf16_tflops": flops / burst_s / 1e12,
            "bf16_tflops_sustained": flops / sustained_s / 1e12,
            "how": "torch: copy of 512 Mi bf16 elements (read + write bytes, best of 10); matmul bf16 8192^3 best of 10 "
                   "(burst) and back to back for %.0f s (sustained)" % seconds}


# ----------------------------------------------------------------------------------------------- CPU oracle arm
class OracleRun:
    """The CPU oracle, as it stands, on the host cores.  One pass = one whole switch_forward + switch_backward of the
    workload over ALL experts (nothing sampled, nothing scaled).  Only the wide-expert workload (8 TFLOP of float64
    matmul per pass) runs the expert FFN on `n_experts` of its experts and scales that part by kept tokens; its
    record says "extrapolated".  Inputs are generated once, outside the timed part."""

    FULL_PASS_FLOP_LIMIT = 3.0e12                              # above this a pass would take minutes on the host

    def __init__(self, cfg: si.SwitchConfig, seed: int, n_experts: int, W_in_bits=None, W_out_bits=None):
        self.cfg = cfg
        self.x, self.dy = si.gen_x(cfg, seed), si.gen_dy(cfg, seed)
        self.W_r, self.b = si.gen_W_r(cfg, seed), si.gen_router_bias(cfg, seed)
        flop = 12.0 * cfg.T * cfg.d_model * cfg.d_ff * (1.5 if cfg.geglu else 1.0)
        self.full = flop <= self.FULL_PASS_FLOP_LIMIT
        self.experts = list(range(cfg.E)) if self.full else list(range(min(max(n_experts, 1), cfg.E)))

        def weights(bits, gen):
            if bits is not None:                               # the same bits the device got, widened to float32
                return {e: si.from_bf16_bits(bits[e]) for e in self.experts}
            return {e: gen(cfg, e, seed) for e in self.experts}

        self.W_in = weights(W_in_bits, si.gen_W_in_expert)
        self.W_out = weights(W_out_bits, si.gen_W_out_expert)
        self.desc, self.kept_all = "", 0

    def step(self) -> float:
        """Seconds of one pass (full) or of one pass scaled to all experts (wide-expert workload only)."""
        from oracle import switch_oracle as so
        cfg, a = self.cfg, (self.x, self.W_r, self.W_in, self.W_out)
        kw = dict(router_bias=self.b, geglu=cfg.geglu)
        if self.full:
            t0 = time.perf_counter()
            fwd = so.switch_forward(*a, cfg.capacity_factor, cfg.alpha, **kw)
            so.switch_backward(fwd, *a, self.dy)
            t = time.perf_counter() - t0
            self.kept_all = int(fwd["kept"].sum())
            self.desc = (f"the whole workload: one switch_forward + switch_backward over all {cfg.T} tokens and all "
                         f"{cfg.E} experts ({self.kept_all} kept tokens), float64 numpy, timed as one pass")
            return t
        t0 = time.perf_counter()
        so.switch_forward(*a, cfg.capacity_factor, cfg.alpha, experts=[], **kw)
        t_rf = time.perf_counter() - t0
        t0 = time.perf_counter()
        fwd = so.switch_forward(*a, cfg.capacity_factor, cfg.alpha, experts=self.experts, **kw)
        t_af = time.perf_counter() - t0
        t0 = time.perf_counter()
        so.switch_backward(fwd, *a, self.dy, experts=self.experts)
        t_ab = time.perf_counter() - t0
        t0 = time.perf_counter()
        so.switch_backward(fwd, *a, self.dy, experts=[])
        t_rb = time.perf_counter() - t0
        kept_sample, self.kept_all = int(fwd["kept"][self.experts].sum()), int(fwd["kept"].sum())
        t_experts = max(t_af - t_rf, 0.0) + max(t_ab - t_rb, 0.0)
        self.desc = (f"EXTRAPOLATED: router+dispatch+loss fwd/bwd on all {cfg.T} tokens; expert FFN fwd+bwd on "
                     f"{len(self.experts)} of {cfg.E} experts ({kept_sample} of {self.kept_all} kept tokens), expert "
                     f"time scaled by kept tokens (a full pass is {12.0 * cfg.T * cfg.d_model * cfg.d_ff / 1e12:.1f} "
                     f"TFLOP of float64 matmul)")
        return t_rf + t_rb + t_experts * self.kept_all / max(kept_sample, 1)

    @staticmethod
    def cores() -> int:
        try:
            from threadpoolctl import threadpool_info
            return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        except Exception:
            return os.cpu_count() or 1


def run_reference(args, cfg):
    """The reference arm: the CPU oracle.  A step is one whole pass of the workload; warm-up and timed passes are
    capped by wall time (a pass takes seconds on the host), and `steps` is the number of passes actually timed."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    run = OracleRun(cfg, args.seed, args.oracle_experts)
    wall0 = time.perf_counter()
    budget_s = args.reference_seconds
    warm_done = 0
    for _ in range(args.warmup):
        if warm_done >= 1 and time.perf_counter() - wall0 > 0.25 * budget_s:
            break
        run.step()
        warm_done += 1
    per_step = []
    for _ in range(args.steps):
        if per_step and time.perf_counter() - wall0 > budget_s:
            break
        per_step.append(run.step())
    t = max(statistics.mean(per_step), 1e-12)
    value = cfg.T / t
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": len(per_step),
        "steps_requested": args.steps, "warmup": warm_done, "warmup_requested": args.warmup,
        "ms_per_step": t * 1e3, "ms_per_step_each": [v * 1e3 for v in per_step],
        "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "T": cfg.T, "d_model": cfg.d_model, "d_ff": cfg.d_ff, "E": cfg.E,
                   "capacity_factor": cfg.capacity_factor, "alpha": cfg.alpha},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": run.cores(), "kind": "oracle", "sample": run.desc,
                         "extrapolated": not run.full},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
        "note": f"passes capped at {budget_s:.0f} s of wall time: `steps` and `warmup` are the passes actually run",
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------- clocks sampler
class ClockSampler:
    """SM clock, power and throttle reasons of one GPU while the timed region runs: NVML polled every 2 ms from a
    thread (read-only queries); nvidia-smi's own loop as the fall-back where NVML cannot be loaded."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    REASON_BITS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}

    def __init__(self, gpu_index: int, pci_bus_id: str | None = None):
        self.rows, self.proc, self.thread = [], None, None
        self.gpu_index, self.pci_bus_id = gpu_index, pci_bus_id
        self.nvml, self.handle, self.stop_flag, self.source = None, None, threading.Event(), "nvidia-smi"
        self.sm, self.power, self.reason_mask, self.sm_max = [], [], 0, None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self.handle = (pynvml.nvmlDeviceGetHandleByPciBusId(self.pci_bus_id.encode()) if self.pci_bus_id
                           else pynvml.nvmlDeviceGetHandleByIndex(self.gpu_index))
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.nvml, self.source = pynvml, "nvml"
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _poll(self):
        n = self.nvml
        while not self.stop_flag.is_set():
            try:
                self.sm.append(float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM)))
                self.power.append(n.nvmlDeviceGetPowerUsage(self.handle) / 1000.0)
                self.reason_mask |= int(n.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
            except Exception:
                pass
            time.sleep(0.002)

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.nvml is not None:
            self.stop_flag.set()
            self.thread.join(timeout=2)
            reasons = sorted(k for k, bit in self.REASON_BITS.items() if self.reason_mask & bit)
            return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_min_mhz": min(self.sm) if self.sm else None,
                    "sm_max_mhz": self.sm_max, "power_w_max": max(self.power) if self.power else None,
                    "samples": len(self.sm), "reasons": reasons, "source": "nvml, polled every 2 ms"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0])); smax.append(float(r[1])); power.append(float(r[2]))
            except ValueError:
                continue
            for n, v in zip(names, r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons),
                "source": "nvidia-smi -lms 100"}


# ----------------------------------------------------------------------------------------------- GPU arm
def run_ours(args, cfg):
    import torch
    from paper_2101_03961_b200 import build as sbuild
    from paper_2101_03961_b200 import switch_moe as sm

    from paper_2101_03961_b200.replicas import Replicas
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the layer has no CPU fallback")
    torch.cuda.set_device(local_rank)
    reps = Replicas("nccl", torch.device("cuda", local_rank))
    rank, world = reps.rank, reps.world
    sbuild.build()
    sm.load_library()

    def dev(a):
        if cfg.dtype == si.DTYPE_BF16:
            return torch.from_numpy(si.to_bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16).reshape(a.shape)
        return torch.from_numpy(a).cuda()

    seed = args.seed + rank                                   # each replica routes its own batch
    x_np, dy_np = si.gen_x(cfg, seed), si.gen_dy(cfg, seed)
    as_bits = cfg.dtype == si.DTYPE_BF16
    W_in_bits = si.gen_W_in(cfg, args.seed, as_bits=as_bits, threads=16)
    W_out_bits = si.gen_W_out(cfg, args.seed, as_bits=as_bits, threads=16)
    if as_bits:
        W_in = torch.from_numpy(W_in_bits.view(np.int16)).cuda().view(torch.bfloat16)
        W_out = torch.from_numpy(W_out_bits.view(np.int16)).cuda().view(torch.bfloat16)
    else:
        W_in, W_out = torch.from_numpy(W_in_bits).cuda(), torch.from_numpy(W_out_bits).cuda()
    x, dy = dev(x_np), dev(dy_np)
    W_r = torch.from_numpy(si.gen_W_r(cfg, args.seed)).cuda()
    b_np = si.gen_router_bias(cfg, args.seed)
    bias = None if b_np is None else torch.from_numpy(b_np).cuda()

    mcfg = sm.make_config(cfg.T, cfg.d_model, cfg.d_ff, cfg.E, cfg.capacity_factor, cfg.alpha, dtype=cfg.dtype,
                          residual=args.residual, groups=args.groups, reroute=args.reroute,
                          reroute_stages=args.reroute_stages, input_jitter=args.input_jitter > 0.0, geglu=cfg.geglu, top2=args.top2,
                          expert_dropout=args.expert_dropout if args.expert_dropout > 0.0 else None)
    noise = None
    if args.router_noise > 0.0:                              # exploration noise on the logits: an input of the layer
        noise = torch.from_numpy(si.gen_router_noise(cfg, args.router_noise, seed)).cuda()
        mcfg.router_noise = noise.data_ptr()
    keep_bits = None
    if args.expert_dropout > 0.0:                            # expert dropout: the keep mask is a seeded input as well
        rows = cfg.E * sm.switch_moe_capacity(mcfg) * max(args.groups, 1)
        keep_bits = torch.from_numpy(si.pack_keep_bits(si.gen_expert_keep(cfg, rows, args.expert_dropout, seed))
                                     .view(np.int32)).cuda()
        mcfg.expert_keep = keep_bits.data_ptr()
    jitter = None
    if args.input_jitter > 0.0:                              # multiplicative jitter on the router's input: an input too
        jitter = dev(si.gen_router_jitter(cfg, args.input_jitter, seed))
        mcfg.router_jitter = jitter.data_ptr()
    ws = sm.allocate_workspace(mcfg)
    y, dx = torch.empty_like(x), torch.empty_like(x)
    dW_in, dW_out, dW_r = torch.empty_like(W_in), torch.empty_like(W_out), torch.empty_like(W_r)
    aux = torch.zeros(1, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        sm.switch_moe_fwd(mcfg, x, W_r, bias, W_in, W_out, y, aux, ws, stream)
        sm.switch_moe_bwd(mcfg, dy, 1.0, x, W_r, W_in, W_out, y, ws, dx, dW_r, dW_in, dW_out, stream)

    def barrier():
        reps.barrier()
        torch.cuda.synchronize()

    props = torch.cuda.get_device_properties(local_rank)
    bus_id = (f"{props.pci_domain_id:08x}:{props.pci_bus_id:02x}:{props.pci_device_id:02x}.0"
              if hasattr(props, "pci_bus_id") else None)           # NVML's index need not be CUDA's

    def measure(n_steps: int, n_warm: int, n_staged: int, n_single: int):
        """`n_warm` untimed steps, then three device-timed regions under one clock sampler: `n_steps` steps with
        nothing recorded between kernels (the library launches its kernels with programmatic dependent launch; an
        event between two kernels would serialise them) -- the step time; `n_staged` steps with the library
        recording an event before every stage -- per-kernel durations for the roofline object and the stage table;
        `n_single` steps with one event per step -- the spread of single steps."""
        for _ in range(n_warm):
            step()
        sm.switch_moe_check_device_status(mcfg, ws, stream)
        events = [[torch.cuda.Event(enable_timing=True) for _ in range(sm.STAGE_EVENTS)] for _ in range(n_staged)]
        for evs in events:
            for ev in evs:
                ev.record(stream)                             # creates the underlying cudaEvent_t handles
        t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler = ClockSampler(local_rank, bus_id)
        barrier()
        sampler.start()
        t_start.record(stream)
        host_t0 = time.perf_counter()
        for _ in range(n_steps):
            step()
        host_ms = (time.perf_counter() - host_t0) * 1e3 / n_steps
        t_end.record(stream)
        barrier()
        ts_start, ts_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ts_start.record(stream)
        for k in range(n_staged):
            sm.set_stage_events(mcfg, events[k])
            step()
        ts_end.record(stream)
        barrier()
        clocks = sampler.stop()
        sm.set_stage_events(mcfg, None)
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(n_single + 1)]
        marks[0].record(stream)
        for k in range(n_single):
            step()
            marks[k + 1].record(stream)
        barrier()
        single = [marks[k].elapsed_time(marks[k + 1]) for k in range(n_single)]
        sm.switch_moe_check_device_status(mcfg, ws, stream)
        ms = reps.max_over_ranks(t_start.elapsed_time(t_end)) / n_steps
        stage_ms = {}
        for i, name in enumerate(sm.STAGE_NAMES):
            if name is not None:
                stage_ms[name] = statistics.mean(events[k][i].elapsed_time(events[k][i + 1]) for k in range(n_staged))
        return {"ms_per_step": ms, "stage_ms": stage_ms, "clocks": clocks, "host_enqueue_ms": host_ms,
                "staged_ms_per_step": ts_start.elapsed_time(ts_end) / n_staged, "single": single}

    # the headline region: exactly K timed steps after W (at least 3) warm-up steps
    head = measure(args.steps, max(args.warmup, 3), args.steps, args.steps)
    ms_per_step, stage_ms, clocks = head["ms_per_step"], head["stage_ms"], head["clocks"]
    host_enqueue_ms, staged_ms_per_step, single = head["host_enqueue_ms"], head["staged_ms_per_step"], head["single"]
    value = reps.tokens_per_second(cfg.T, ms_per_step)
    # A run of a few dozen steps is over before the 1000 W power cap pulls the SM clock down (the burst state); a
    # run of hundreds of steps sits at the capped clock.  A short run therefore appends a sustained region (300
    # warm-up steps, 300 timed, 100 with stage events) so that its line carries both states.
    sustained_run = None
    if args.steps < 200 and not args.no_sustained:
        sustained_run = measure(300, 300, 100, 20)

    if not reps.is_reporting_rank:
        reps.close()
        return

    kept_per_expert = sm.switch_moe_workspace_view(mcfg, ws, sm.WS_KEPT)
    kept = int(kept_per_expert.sum().item())
    busy = float((kept_per_expert > 0).sum().item()) / cfg.E   # experts without tokens: their weights are never read
    peaks, peak_kind = load_peaks()
    hbm = float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))
    elt = 2 if cfg.dtype == si.DTYPE_BF16 else 4
    row_bytes = cfg.d_model * elt
    gemm_names = ["gemm1_relu", "gemm2_combine", "dgrad2_mask", "wgrad2", "dgrad1_scatter", "wgrad1"]
    # useful flops of one expert GEMM (kept rows only); with GEGLU experts the three GEMMs that touch W_in have twice
    # the columns, and the figure is the mean over the six products
    gemm_weight = {n: 1.0 for n in gemm_names}
    if cfg.geglu:
        gemm_weight.update({"gemm1_relu": 2.0, "dgrad1_scatter": 2.0, "wgrad1": 2.0})
    flops_unit = 2.0 * kept * cfg.d_model * cfg.d_ff
    flops_per_launch = flops_unit * sum(gemm_weight.values()) / 6.0
    # Algorithmic DRAM bytes of one product, mean over the six: its expert weights once (read -- only of experts
    # that kept a token -- or written for a weight gradient: every expert's, zeros included) and its two activation
    # operands once, over kept rows only (d-wide rows: X_d, dY_d, y, dx;
    # f-wide rows: H, dH), plus the one-bit ReLU mask written by GEMM1 and read by dgrad2.
    fin = cfg.d_ff * (2 if cfg.geglu else 1)
    w_in_b, w_out_b = cfg.E * cfg.d_model * fin * elt, cfg.E * cfg.d_ff * cfg.d_model * elt
    rows_d, rows_f, rows_fin = kept * cfg.d_model * elt, kept * cfg.d_ff * elt, kept * fin * elt
    mask_b = 0 if cfg.geglu else kept * cfg.d_ff // 8
    algo_bytes = {"gemm1_relu": busy * w_in_b + rows_d + rows_fin + mask_b,
                  "gemm2_combine": busy * w_out_b + rows_f + rows_d,
                  "dgrad2_mask": busy * w_out_b + rows_d + rows_f + mask_b, "wgrad2": w_out_b + rows_f + rows_d,
                  "dgrad1_scatter": busy * w_in_b + rows_fin + rows_d, "wgrad1": w_in_b + rows_d + rows_fin}
    traffic_algorithmic = sum(algo_bytes.values()) / 6.0
    captured = load_captured_traffic(cfg)

    def roofline_of(st_ms, clk):
        gemm_ms_avg = statistics.mean(st_ms[n] for n in gemm_names)
        achieved_tf = flops_per_launch / (gemm_ms_avg * 1e-3) / 1e12
        if cfg.dtype != si.DTYPE_BF16:
            peak_tf = 148 * 128 * 2 * 1.965e9 / 1e12
            return {"bound": "alu", "kernel": "simt_grouped_gemm_kernel", "achieved": achieved_tf, "peak": peak_tf,
                    "unit": "TFLOP/s", "frac": achieved_tf / peak_tf, "traffic": None,
                    "peak_source": "148 SMs x 128 FP32 lanes x 2 x 1.965 GHz"}
        # Which measured peak the launches are held against depends on the state the GPU was timed in: the burst
        # figure before the power cap pulls the SM clock down, the sustained figure at the capped clock.  The
        # sampled clocks decide; without samples the larger (burst) peak is used.
        sm_med, sm_top = (clk or {}).get("sm_mhz"), (clk or {}).get("sm_max_mhz")
        capped = bool(sm_med and sm_top and sm_med < 0.9 * sm_top)
        peak_key = "bf16_tflops_sustained" if capped else "bf16_tflops"
        peak_tf = float(peaks.get(peak_key, FALLBACK_PEAKS[peak_key]))
        traffic = captured["bytes_per_product"] if captured else None
        algo_gbs = traffic_algorithmic / (gemm_ms_avg * 1e-3) / 1e9
        return {"bound": "tensor",
                "kernel": "expert_gemm_pair_kernel (6 products per step in 5 launches, mean per product)",
                "achieved": achieved_tf, "peak": peak_tf, "unit": "TFLOP/s", "frac": achieved_tf / peak_tf,
                "traffic": traffic,
                "traffic_source": captured["source"] if captured else
                "no ncu capture recorded for this shape (profiles/expert_gemm_dram_traffic.txt): null",
                "traffic_algorithmic": traffic_algorithmic,
                "peak_source": (f"{peak_kind} bf16 sustained (timed at the power-capped clock, median {sm_med} MHz)"
                                if capped else
                                f"{peak_kind} bf16 burst (timed before the power cap set in, median {sm_med} MHz)"),
                "frac_of_sustained_peak": achieved_tf / float(peaks.get("bf16_tflops_sustained",
                                                                    FALLBACK_PEAKS["bf16_tflops_sustained"])),
                "flops_per_launch": flops_per_launch, "avg_launch_ms": gemm_ms_avg,
                "frac_of_burst_peak": achieved_tf / float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"])),
                # the same launches against the copy bandwidth, from the algorithmic bytes and this run's times
                "hbm_gbs_algorithmic": algo_gbs, "hbm_frac_algorithmic": algo_gbs / hbm,
                "time_x_clock_ms_mhz": None if not sm_med else gemm_ms_avg * sm_med,
                # nominal figures for context: 2250 TFLOP/s dense bf16, 8000 GB/s HBM3e
                "frac_of_nominal_peak": achieved_tf / 2250.0, "hbm_frac_of_nominal": algo_gbs / 8000.0}

    def stages_of(st_ms):
        stages = {n: {"ms": st_ms[n]} for n in st_ms}
        for n in gemm_names:
            stages[n]["tflops"] = flops_unit * gemm_weight[n] / (st_ms[n] * 1e-3) / 1e12
            stages[n]["hbm_frac"] = algo_bytes[n] / (st_ms[n] * 1e-3) / 1e9 / hbm
        if cfg.dtype == si.DTYPE_BF16:
            # the two products of dH run as one launch: the event between them falls after both
            both = st_ms["dgrad1_scatter"] + st_ms["wgrad1"]
            del stages["wgrad1"]
            del stages["dgrad1_scatter"]
            stages["dgrad1_scatter+wgrad1"] = {
                "ms": both,
                "tflops": flops_unit * (gemm_weight["dgrad1_scatter"] + gemm_weight["wgrad1"]) / (both * 1e-3) / 1e12,
                "hbm_frac": (algo_bytes["dgrad1_scatter"] + algo_bytes["wgrad1"] - rows_fin) / (both * 1e-3) / 1e9 / hbm}
        probs_b = cfg.T * cfg.E * 4
        stages["gather_x"]["gbs"] = (2 * kept * row_bytes) / (st_ms["gather_x"] * 1e-3) / 1e9
        stages["gather_dy"]["gbs"] = (3 * kept * row_bytes) / (st_ms["gather_dy"] * 1e-3) / 1e9
        stages["router_fwd"]["gbs"] = (cfg.T * row_bytes + probs_b) / (st_ms["router_fwd"] * 1e-3) / 1e9
        # router backward: reads x, the probabilities and dx, writes dx (dW_r and the per-token vectors are small)
        stages["router_bwd"]["gbs"] = (3 * cfg.T * row_bytes + probs_b) / (st_ms["router_bwd"] * 1e-3) / 1e9
        stages["router_fwd"]["fp32_tflops"] = 2.0 * cfg.T * cfg.d_model * cfg.E / (st_ms["router_fwd"] * 1e-3) / 1e12
        stages["router_bwd"]["fp32_tflops"] = 4.0 * cfg.T * cfg.d_model * cfg.E / (st_ms["router_bwd"] * 1e-3) / 1e12
        for n in ("gather_x", "gather_dy", "router_fwd", "router_bwd"):
            stages[n]["hbm_frac"] = stages[n]["gbs"] / hbm
        per_stage = sm.switch_moe_stage_launches(mcfg)
        for n, st in stages.items():
            st["launches"] = (per_stage["dgrad1_scatter"] + per_stage["wgrad1"] if n == "dgrad1_scatter+wgrad1"
                              else per_stage[n])
            st["us_per_launch"] = st["ms"] * 1e3 / max(st["launches"], 1)
        return stages

    roofline = roofline_of(stage_ms, clocks)
    stages = stages_of(stage_ms)
    sustained = None
    if sustained_run is not None:
        r2 = roofline_of(sustained_run["stage_ms"], sustained_run["clocks"])
        sustained = {"ms_per_step": sustained_run["ms_per_step"],
                     "value": reps.tokens_per_second(cfg.T, sustained_run["ms_per_step"]),
                     "steps": 300, "warmup": 300, "sm_mhz": (sustained_run["clocks"] or {}).get("sm_mhz"),
                     "reasons": (sustained_run["clocks"] or {}).get("reasons"),
                     "roofline_frac": r2["frac"], "roofline_peak": r2["peak"], "roofline_achieved": r2["achieved"],
                     "roofline_peak_source": r2["peak_source"], "avg_gemm_launch_ms": r2.get("avg_launch_ms"),
                     "hbm_frac_algorithmic": r2.get("hbm_frac_algorithmic"),
                     "time_x_clock_ms_mhz": r2.get("time_x_clock_ms_mhz"),
                     "stages_ms": {k: v["ms"] for k, v in stages_of(sustained_run["stage_ms"]).items()},
                     "single_steps_ms": {"median": statistics.median(sustained_run["single"])}}

    # ---- end to end through the C ABI with HOST activations (pinned), copies inside the timed region
    xh, dyh = x.cpu().pin_memory(), dy.cpu().pin_memory()
    yh, dxh = torch.empty_like(xh).pin_memory(), torch.empty_like(xh).pin_memory()
    auxh = torch.zeros(1).pin_memory()
    e2e_steps = max(2, min(args.steps, 10))

    up_stream, down_stream = torch.cuda.Stream(), torch.cuda.Stream()

    def host_step():
        sm.switch_moe_step_host(mcfg, xh, dyh, 1.0, W_r, bias, W_in, W_out, x, dy, y, dx, aux, dW_r, dW_in, dW_out,
                                yh, dxh, auxh, ws, stream, up_stream, down_stream)

    host_step()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        host_step()                                           # synchronises the stream before returning
    blocking_s = (time.perf_counter() - t0) / e2e_steps

    # the same step kept two deep with the non-blocking call: step i + 1 uploads while step i computes and step i - 1
    # downloads; every step still copies its own inputs in and its own results out
    slots = []
    for _ in range(2):
        slots.append({"x": torch.empty_like(x), "dy": torch.empty_like(dy), "y": torch.empty_like(y),
                      "dx": torch.empty_like(dx), "aux": torch.zeros(1, device="cuda"),
                      "yh": torch.empty_like(xh).pin_memory(), "dxh": torch.empty_like(xh).pin_memory(),
                      "auxh": torch.zeros(1).pin_memory(), "done": None})

    def pipelined(n):
        for i in range(n):
            sl = slots[i % 2]
            done = torch.cuda.Event()
            sm.switch_moe_step_host_enqueue(mcfg, xh, dyh, 1.0, W_r, bias, W_in, W_out, sl["x"], sl["dy"], sl["y"],
                                            sl["dx"], sl["aux"], dW_r, dW_in, dW_out, sl["yh"], sl["dxh"], sl["auxh"],
                                            ws, stream, up_stream, down_stream, sl["done"], done)
            sl["done"] = done
        for sl in slots:
            if sl["done"] is not None:
                sl["done"].synchronize()

    pipelined(2)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    pipelined(e2e_steps)
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    sm.switch_moe_check_device_status(mcfg, ws, stream)
    assert torch.equal(slots[0]["yh"], yh) and torch.equal(slots[1]["dxh"], dxh)   # same results as the blocking call
    act_bytes = cfg.T * row_bytes
    e2e = {"value": world * cfg.T / e2e_s, "unit": UNIT, "h2d_bytes_per_step": 2 * act_bytes,
           "d2h_bytes_per_step": 2 * act_bytes + 4, "ms_per_step": e2e_s * 1e3,
           "pcie_gbs_each_way": 2 * act_bytes / e2e_s / 1e9,   # both directions carry this at once
           "blocking_call_value": world * cfg.T / blocking_s, "blocking_call_ms_per_step": blocking_s * 1e3,
           "note": "switch_moe_step_host_enqueue, two steps in flight: every step copies x, dy from pinned host memory "
                   "and y, dx, aux back; weights and weight gradients resident.  blocking_call_*: switch_moe_step_host, "
                   "one step at a time (dy upload overlaps forward, y download overlaps backward)"}

    # ---- CPU baseline: the oracle, whole workload, on this machine's host cores (one warm-up pass, one timed pass)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        orun = OracleRun(cfg, args.seed, args.oracle_experts, W_in_bits if as_bits else None,
                         W_out_bits if as_bits else None)
        orun.step()                                           # warm-up (BLAS threads, page faults)
        t = orun.step()
        cpu = {"value": cfg.T / t, "unit": UNIT, "cores": orun.cores(), "kind": "oracle", "sample": orun.desc,
               "seconds": t, "extrapolated": not orun.full}
    del W_in_bits, W_out_bits

    # ---- this box's own copy bandwidth and bf16 matmul rate, measured now (context for the fractions above)
    box = None
    if not args.no_box_peaks:
        box = same_run_peaks(torch.device("cuda", local_rank))
        if roofline.get("bound") == "tensor":
            roofline["frac_of_same_run_sustained"] = roofline["achieved"] / box["bf16_tflops_sustained"]
            roofline["frac_of_same_run_burst"] = roofline["achieved"] / box["bf16_tflops"]
            roofline["hbm_frac_algorithmic_of_same_run_copy"] = roofline["hbm_gbs_algorithmic"] / box["hbm_gbs"]

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.dtype == si.DTYPE_BF16 else "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "T": cfg.T, "d_model": cfg.d_model, "d_ff": cfg.d_ff, "E": cfg.E,
                   "geglu_experts": cfg.geglu,
                   "capacity_factor": cfg.capacity_factor, "alpha": cfg.alpha, "capacity": sm.switch_moe_capacity(mcfg),
                   "kept_tokens": kept, "parallelism": "replicas" if world > 1 else "single",
                   "skip_path_inside_layer": bool(args.residual), "routing_groups": args.groups, "reroute_overflow": bool(args.reroute), "reroute_stages": args.reroute_stages if args.reroute else 0, "top2_routing": bool(args.top2), "expert_dropout": args.expert_dropout, "router_noise_eps": args.router_noise, "input_jitter_eps": args.input_jitter,
                   "l2": "inputs larger than L2 (weights 2 x %.0f MB per pass), no flush" %
                         (cfg.E * cfg.d_model * cfg.d_ff * elt / 1e6)},
        "clocks": clocks, "e2e": e2e, "gpu_launches": sm.switch_moe_launches_per_step(mcfg) * args.steps,
        "roofline": roofline, "cpu_baseline": cpu, "stages": stages, "host_enqueue_ms_per_step": host_enqueue_ms,
        "ms_per_step_with_stage_events": staged_ms_per_step,
        "box_peaks_same_run": box,
        "single_steps_ms": {"median": statistics.median(single), "best": min(single), "worst": max(single)},
        "sustained": sustained if sustained is not None else "the headline region itself ran %d steps after %d" %
                                                              (args.steps, max(args.warmup, 3)),
        "aux_loss": float(aux.item()),
    }
    print(json.dumps(line), flush=True)
    reps.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    # defaults (300 warm-up, 500 timed steps): long enough for the GPU to settle at its power-capped clock before the
    # timed steps (about 0.4 s of warm-up) and to average over the cap's swings (0.7 s per timed region), so that the
    # default line is a sustained figure; the whole run still takes seconds
    # (the reference arm's steps take seconds each on the host: its defaults are 3 timed steps after 1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="switch_base", choices=sorted(si.CONFIGS))
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--oracle-experts", type=int, default=None,
                    help="experts whose FFN the CPU oracle runs in its bounded sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sustained", action="store_true",
                    help="skip the sustained region (300 warm-up + 300 timed steps) that a run of fewer than 200 "
                         "steps appends to its line")
    ap.add_argument("--reference-seconds", type=float, default=150.0,
                    help="wall-time cap of the reference arm's passes (each pass is the whole workload on the host)")
    ap.add_argument("--no-box-peaks", action="store_true",
                    help="skip the torch copy / bf16 matmul measurement of this box at the end of the run")
    ap.add_argument("--groups", type=int, default=1,
                    help="route the batch as this many independent groups of T / groups tokens (own capacity and "
                         "loss each, experts shared); the headline configuration is one group")
    ap.add_argument("--router-noise", type=float, default=0.0,
                    help="add uniform(1 - eps, 1 + eps) noise (a seeded input tensor) to the router logits; "
                         "the headline configuration has none")
    ap.add_argument("--input-jitter", type=float, default=0.0,
                    help="multiply the router's input by uniform(1 - eps, 1 + eps) factors (a seeded input tensor); "
                         "the headline configuration has none")
    ap.add_argument("--top2", action="store_true",
                    help="top-2 routing (the Mixture-of-Experts comparator): two assignments per token, so about twice "
                         "the expert work of the headline configuration at a capacity factor that keeps them")
    ap.add_argument("--expert-dropout", type=float, default=0.0,
                    help="dropout rate on the experts' hidden activations (fine-tuning regularisation; seeded keep mask)")
    ap.add_argument("--reroute", action="store_true",
                    help="offer tokens that overflow their expert to their second choice (stage 2 of "
                         "No-Token-Left-Behind routing); not the headline configuration")
    ap.add_argument("--reroute-stages", type=int, default=1,
                    help="with --reroute: how many stages follow stage 1 (stage k offers the k-th choice)")
    ap.add_argument("--residual", action="store_true",
                    help="time the variant that adds the layer's input to its output inside the combine step "
                         "(y = x + layer(x), dx = dy + ...); not the headline configuration")
    args = ap.parse_args()
    cfg = si.CONFIGS[args.workload]
    if args.steps is None:
        args.steps = 3 if args.impl == "reference" else 500
    if args.warmup is None:
        args.warmup = 1 if args.impl == "reference" else 300
    if args.oracle_experts is None:
        # only the wide-expert workload samples experts (about 3e11 flops of fp64 matmul per pass)
        per_expert = 12.0 * (cfg.T / cfg.E) * cfg.d_model * cfg.d_ff
        args.oracle_experts = int(max(1, min(cfg.E, round(3.0e11 / per_expert))))
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
