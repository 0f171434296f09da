#!/usr/bin/env python
"""MoE-layer benchmark: tokens/s of the whole hot path (route -> dispatch -> expert FFN -> combine).

    python bench.py --gpus N --steps K --warmup W            # the CUDA path
    python bench.py --impl reference --steps K --warmup W    # the CPU oracle, bounded sample per step

A step is one pass of the whole layer over one batch of seeded synthetic input.  At N > 1 (launched
by torch.distributed.run, one process per GPU) every rank runs an independent replica on its own
batch (the path does not shard: weak scaling, no data-path collective); the time is the max over
ranks.  Rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2605_05888_b200 import inputs  # noqa: E402

METRIC = "MoE-layer tokens/s on 1 B200; dispatch+combine HBM GB/s and % of roofline"
UNIT = "tokens/s"
WORKLOADS = {"c1": inputs.C1, "c2": inputs.C2, "c3": inputs.C3, "c4": inputs.C4,
             # a quarter-size C2 (same kernels, 0.7 GB of weights) for ncu captures that must stay small
             "c2_small": inputs.C2.with_(name="mixtral_like_bf16_small", T=2048, E=4, R=4, F=7168),
             # a reduced DeepSeek-V3-like layer (same H, F, top-8 and Zipf bias; 32 experts, 1024 tokens: 2.8 GB of
             # weights) for ncu captures of the expert kernel in its skewed, weight-streaming regime
             "c3_small": inputs.C3.with_(name="deepseek_v3_like_bf16_small", T=1024, E=32, R=4),
             # the other two shapes of the paper's Table II
             "phi35": inputs.PHI35, "qwen64": inputs.QWEN64,
             # dispatch/combine-only sweep points (identity experts)
             "c5_8192": inputs.C5(8192), "c5_8192_zipf": inputs.C5(8192, 1.2), "c5_2048": inputs.C5(2048)}



def ncu_traffic_bytes(workload: str):
    """DRAM traffic of the dominant kernel per step, measured with ncu and kept beside the profile summaries."""
    path = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")
    try:
        with open(path) as f:
            entry = json.load(f).get(workload)
        return None if entry is None else float(entry["bytes"])
    except (OSError, ValueError, KeyError, TypeError):
        return None



def load_peaks() -> tuple[dict, str]:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


def pick_dispatch(args, w: inputs.Workload) -> str:
    """--dispatch auto: the token-ordered bulk-copy scheme where the dispatch moves at least half a gigabyte (there
    it is the fastest: 0.80 of the copy rate against 0.66 on the DeepSeek-like layer), else the paged scheme
    (faster on small batches: one wave of small CTAs)."""
    if args.dispatch != "auto":
        return args.dispatch
    moved = w.T * w.H * w.elem_bytes * (1 + w.K)
    return "ordered" if moved >= 512e6 else "paged"


def workload_config(w: inputs.Workload, extra: dict) -> dict:
    cfg = {"workload": w.name, "T": w.T, "H": w.H, "E": w.E, "R": w.R, "K": w.K, "F": w.F,
           "router": "softmax top-K, zipf_s=%g" % w.zipf_s, "seed": w.seed}
    cfg.update(extra)
    return cfg


# ------------------------------------------------------------------------------------------------
# CPU oracle legs (the only places this file touches oracle/)
def oracle_sample(w: inputs.Workload, n_tokens: int, x, wr, bias, wg, wu, wd) -> tuple[float, int]:
    """Times the oracle layer on the first n_tokens tokens of the batch. Returns (seconds, threads)."""
    import oracle
    xs = np.ascontiguousarray(x[:n_tokens])
    t0 = time.perf_counter()
    if w.identity_experts:
        oracle.layer(xs, wr, bias, None, None, None, w.E, w.R, w.K, w.dtype, identity_experts=True)
    else:
        oracle.layer(xs, wr, bias, list(wg), list(wu), list(wd), w.E, w.R, w.K, w.dtype)
    return time.perf_counter() - t0, oracle.num_threads()


def oracle_sample_tokens(w: inputs.Workload, threads: int) -> int:
    """Tokens whose oracle layer costs roughly 10-20 s on `threads` cores at ~2.5 GFLOP/s per core."""
    flop_per_token = 6.0 * w.K * w.H * max(w.F, 1) + 2.0 * w.H * w.E
    n = int(15.0 * 2.5e9 * max(threads, 1) / flop_per_token)
    return max(8, min(w.T, n))


def run_reference(args, w: inputs.Workload) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    x = inputs.make_x(w)
    wr, bias = inputs.make_router(w)
    wg, wu, wd = inputs.make_all_expert_weights(w) if not w.identity_experts else (None, None, None)
    threads = oracle.num_threads()
    # keep the whole run within a few minutes: (steps + warmup) samples of n tokens each
    n = max(4, oracle_sample_tokens(w, threads) // max(1, (args.steps + args.warmup) // 2))
    for _ in range(args.warmup):
        oracle_sample(w, n, x, wr, bias, wg, wu, wd)
    t = 0.0
    for _ in range(args.steps):
        dt, _ = oracle_sample(w, n, x, wr, bias, wg, wu, wd)
        t += dt
    value = n * args.steps / t
    sample = f"first {n} of {w.T} tokens per step, whole layer (route, dispatch, experts, combine)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(w, {"sample": sample}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self.power_w, self.power_limit_w = [], None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            try:
                self.power_limit_w = pynvml.nvmlDeviceGetEnforcedPowerLimit(self.h) / 1000.0
            except Exception:
                self.power_limit_w = None
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
                 getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                 getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                 getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
                 getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake"}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
                mask = get(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            try:  # board power (NVML averages it over a window of its own, so short runs under-read)
                self.power_w.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
            except Exception:
                pass
            self._stop_evt.wait(0.005)

    def energy_mj(self):
        """The board's energy counter (millijoules since the driver was loaded), or None."""
        try:
            return float(self.nv.nvmlDeviceGetTotalEnergyConsumption(self.h)) if self.ok else None
        except Exception:
            return None

    def stop(self) -> dict:
        self._stop_evt.set()
        if self.is_alive():
            self.join(1.0)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples),
                "power_w_max": (round(max(self.power_w), 1) if self.power_w else None), "power_limit_w": self.power_limit_w}


def plain_copy_us(total_bytes: float) -> float | None:
    """Yardstick for the copy-bound stages: a plain device-to-device copy that moves the same number of bytes
    (half read, half written), timed the way the per-kernel pass times a stage - one launch between two events,
    synchronised - median of 9.  Small stages cannot beat it however they are written."""
    import torch
    try:
        n = max(1, int(total_bytes) // 4)            # bf16 elements: n * 2 bytes read + n * 2 bytes written
        src = torch.empty(n, dtype=torch.bfloat16, device="cuda").normal_()
        dst = torch.empty_like(src)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ts = []
        for i in range(12):
            torch.cuda.synchronize()
            e0.record()
            dst.copy_(src)
            e1.record()
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(e0.elapsed_time(e1) * 1e3)
        return float(np.median(ts))
    except Exception:
        return None


def max_over_ranks(values: list[float], device: str = "cpu") -> list[float]:
    """Element-wise max of per-rank timings over the default process group (identity when single-process)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_tokens_per_s(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Replicas: every rank processes tokens_per_rank tokens per step; time is the max over ranks."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def brief_measurement(args, w: inputs.Workload) -> dict:
    """ms/step, tokens/s and the per-stage figures of one more workload, device-resident inputs only (no host
    copies, no oracle): kept in the main line so that its numbers can be followed from round to round."""
    import torch

    from paper_2605_05888_b200 import binding as B

    def dev(a):
        if a is None:
            return None
        t = torch.from_numpy(a)
        return t.view(torch.int16).cuda().view(torch.bfloat16) if a.dtype == np.uint16 else t.cuda()

    x = inputs.make_x(w)
    wr, bias = inputs.make_router(w)
    wg, wu, wd = inputs.make_all_expert_weights(w)
    t = [dev(a) for a in (x, wr, bias, wg, wu, wd)]
    del wg, wu, wd
    dispatch = pick_dispatch(args, w)
    mode = {"scan": B.DISPATCH_SCAN, "static": B.DISPATCH_ATOMIC_STATIC, "paged": B.DISPATCH_ATOMIC_PAGED,
            "ordered": B.DISPATCH_ATOMIC_ORDERED}[dispatch]
    plan = B.Plan(B.make_config(w.T, w.H, w.E, w.R, w.K, w.F, w.dtype, dispatch_mode=mode))
    y = torch.empty((w.T, w.H), dtype=torch.bfloat16, device="cuda")
    for _ in range(max(args.warmup, 3)):
        plan.moe_layer(*t, y)
    torch.cuda.synchronize()
    plan.moe_ffn_clock_mhz(reset=True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        plan.moe_layer(*t, y)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    clock = round(plan.moe_ffn_clock_mhz(reset=True), 1)
    stage_ms = np.zeros(len(B.STAGES))
    for _ in range(args.steps):
        stage_ms += np.array(plan.moe_layer_timed(*t, y))
    sm = dict(zip(B.STAGES, (stage_ms / args.steps).tolist()))
    code, detail = plan.moe_last_status()
    if code != 0:
        return {"error": f"device status {code}, detail {detail}"}
    peaks, _ = load_peaks()
    eb, rows = w.elem_bytes, w.T * w.K
    flops = 6.0 * rows * w.H * w.F
    t_ffn = sm["gemm1"] + sm["gemm2"]
    disp_b, comb_b = w.T * w.H * eb * (1 + w.K) + 12 * rows, w.T * w.H * eb * (w.K + 1) + 8 * rows
    disp = disp_b / sm["dispatch"] / 1e6
    comb = comb_b / sm["combine"] / 1e6
    copy_us = plain_copy_us(disp_b)
    return {"ms_per_step": ms, "value": w.T / ms * 1e3, "unit": UNIT, "steps": args.steps,
            "config": workload_config(w, {"dispatch_mode": dispatch}),
            "ffn": {"ms": t_ffn, "TFLOPs": flops / t_ffn / 1e9, "frac_of_burst_peak": flops / t_ffn / 1e9 / peaks["bf16_tflops"],
                    "kernel_sm_mhz": clock},
            "route_ms": sm["route"],
            "dispatch": {"ms": sm["dispatch"], "GBps": disp, "frac_hbm": disp / peaks["hbm_gbs"], "plain_copy_same_bytes_us": copy_us,
                         "time_vs_plain_copy": (sm["dispatch"] * 1e3 / copy_us) if copy_us else None},
            "combine": {"ms": sm["combine"], "GBps": comb, "frac_hbm": comb / peaks["hbm_gbs"], "plain_copy_same_bytes_us": copy_us,
                        "time_vs_plain_copy": (sm["combine"] * 1e3 / copy_us) if copy_us else None},
            "stages_from": "a separate pass with an event after every kernel and a synchronisation per step"}


def run_cuda(args, w: inputs.Workload) -> None:
    import torch
    import torch.distributed as dist

    from paper_2605_05888_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no CPU fallback (use --impl reference)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    w = w.with_(seed=w.seed + rank)  # every rank its own batch

    def dev(a):
        if a is None:
            return None
        t = torch.from_numpy(a)
        return t.view(torch.int16).cuda().view(torch.bfloat16) if a.dtype == np.uint16 else t.cuda()

    x = inputs.make_x(w)
    wr, bias = inputs.make_router(w)
    if w.identity_experts:
        wg = wu = wd = None
    else:
        wg, wu, wd = inputs.make_all_expert_weights(w.with_(seed=0))  # same parameters on every rank
    dx, dwr, dbias, dwg, dwu, dwd = dev(x), dev(wr), dev(bias), dev(wg), dev(wu), dev(wd)
    el = torch.bfloat16 if w.dtype == inputs.BF16 else torch.float32
    dispatch = pick_dispatch(args, w)
    mode = {"scan": B.DISPATCH_SCAN, "static": B.DISPATCH_ATOMIC_STATIC, "paged": B.DISPATCH_ATOMIC_PAGED,
            "ordered": B.DISPATCH_ATOMIC_ORDERED}[dispatch]
    plan = B.Plan(B.make_config(w.T, w.H, w.E, w.R, w.K, w.F, w.dtype, dispatch_mode=mode,
                                identity_experts=int(w.identity_experts), ffn_split=int(args.ffn_split),
                                ffn_kernel=args.ffn_kernel, ffn_hot_min_tiles=args.ffn_hot_min_tiles, ffn_thin_tiles=args.ffn_thin_tiles, route_filter=args.route_filter,
                                overlap=args.overlap, combine_mode=args.combine_mode, tp_shards=args.tp_shards))
    y = torch.empty((w.T, w.H), dtype=el, device="cuda")
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def step():
        plan.moe_layer(dx, dwr, dbias, dwg, dwu, dwd, y)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    code, detail = plan.moe_last_status()
    if code != 0:
        raise SystemExit(f"bench.py: device status {code} ({B.strerror(code)}), detail {detail}")
    launches_per_step = plan.moe_last_launch_count()

    # ---- timed region: K steps, device-resident inputs ----
    sampler = ClockSampler(local)
    barrier()
    plan.moe_ffn_clock_mhz(reset=True)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    mj0 = sampler.energy_mj()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    mj1 = sampler.energy_mj()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop()
    if mj0 is not None and mj1 is not None and mj1 > mj0 and ms_total >= 800.0:
        # NVML's energy counter over the timed region: joules per layer and the mean board power they imply.  The
        # counter advances in steps of some tens of milliseconds and lags, so only regions of about a second or
        # more are reported (--steps 150 or so on the default workload).
        clocks["energy_j_per_step"] = round((mj1 - mj0) / 1e3 / args.steps, 3)
        clocks["mean_power_w"] = round((mj1 - mj0) / ms_total, 1)
    # SM clock the tensor-core expert kernel really ran at (cycles / time measured inside the kernel): THE clock
    # of the dominant kernel.  sm_mhz is what NVML returned when polled every 5 ms during the timed region; a
    # region of tens of milliseconds gives it a handful of samples, taken mostly between kernels.
    clocks["ffn_kernel_sm_mhz"] = round(plan.moe_ffn_clock_mhz(reset=True), 1)
    clocks["sm_mhz_is"] = "NVML samples (see samples); the dominant kernel's own clock is ffn_kernel_sm_mhz"
    barrier()

    # ---- per-kernel device times: the same steps with an event after every kernel ----
    stage_ms = np.zeros(len(B.STAGES))
    for _ in range(args.steps):
        stage_ms += np.array(plan.moe_layer_timed(dx, dwr, dbias, dwg, dwu, dwd, y))
    stage_ms /= args.steps

    # ---- availability timeline of the dispatch (when does each 128-row tile become ready): 5 traced layers ----
    plan.moe_availability_trace(True)
    for _ in range(5):
        step()
    torch.cuda.synchronize()
    trace = plan.layer_tensor(8).cpu().numpy().astype(np.float64)
    plan.moe_availability_trace(False)
    ready = trace[2:][trace[2:] > 0] - trace[0]
    availability = {"full_tiles": int(ready.size), "all_ready_us": (trace[1] - trace[0]) / 1e3,
                    "first_full_tile_us": float(ready.min() / 1e3) if ready.size else None,
                    "median_full_tile_us": float(np.median(ready) / 1e3) if ready.size else None,
                    "last_full_tile_us": float(ready.max() / 1e3) if ready.size else None,
                    "what": "microseconds after the first dispatch CTA started (device %globaltimer), one traced layer"}

    # ---- the overlapped launch (dispatch inside the expert kernel's launch), measured beside the main plan ----
    overlap_arm = None
    if rank == 0 and world == 1 and args.overlap == 0 and w.dtype == inputs.BF16 and not w.identity_experts \
            and args.ffn_kernel == 0 and args.tp_shards <= 1:
        try:
            po = B.Plan(B.make_config(w.T, w.H, w.E, w.R, w.K, w.F, w.dtype, dispatch_mode=B.DISPATCH_ATOMIC_ORDERED,
                                      ffn_split=int(args.ffn_split), overlap=1, combine_mode=args.combine_mode))
            for _ in range(3):
                po.moe_layer(dx, dwr, dbias, dwg, dwu, dwd, y, stream)
            torch.cuda.synchronize()
            n_ov = min(args.steps, 10)
            e0.record()
            for _ in range(n_ov):
                po.moe_layer(dx, dwr, dbias, dwg, dwu, dwd, y, stream)
            e1.record()
            torch.cuda.synchronize()
            po.moe_availability_trace(True)
            po.layer_tensor(9).zero_()
            po.moe_layer(dx, dwr, dbias, dwg, dwu, dwd, y, stream)
            torch.cuda.synchronize()
            tr = po.layer_tensor(8).cpu().numpy().astype(np.float64)
            items = po.layer_tensor(9).cpu().numpy()
            po.moe_availability_trace(False)
            started = items[items[:, 0] > 0]
            g1 = started[(started[:, 2] & 1) == 0]
            rdy = tr[2:][tr[2:] > 0] - tr[0]
            code_o, _ = po.moe_last_status()
            overlap_arm = {"ms_per_step": e0.elapsed_time(e1) / n_ov, "steps": n_ov, "status": code_o,
                           "all_ready_us": (tr[1] - tr[0]) / 1e3,
                           "first_full_tile_us": float(rdy.min() / 1e3) if rdy.size else None,
                           "first_gemm1_item_start_us": float((g1[:, 0].min() - tr[0]) / 1e3) if g1.size else None,
                           "what": "overlap = 1: producer CTAs run the ordered dispatch inside the expert launch, consumer CTAs "
                                   "start a tile when its status counter is full; times after the first dispatch CTA started"}
            del po
        except Exception as exc:  # measurement beside the main line: never takes the line down
            overlap_arm = {"error": str(exc)[:200]}

    # ---- end to end through the host-buffer entry point: H2D of x and D2H of y inside the timing ----
    hx = torch.from_numpy(x.view(np.int16) if x.dtype == np.uint16 else x).pin_memory()
    hy = torch.empty_like(hx).pin_memory()
    for _ in range(3):
        plan.moe_layer_host(hx, dwr, dbias, dwg, dwu, dwd, hy)
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        plan.moe_layer_host(hx, dwr, dbias, dwg, dwu, dwd, hy)   # returns when h_y is complete
    ms_e2e_sync = 1e3 * (time.perf_counter() - t0)
    # the pipelined form: two steps in flight, every step still copies its x in and its y out
    hx2, hy2 = [hx, hx.clone().pin_memory()], [hy, torch.empty_like(hy).pin_memory()]
    tickets = []
    for i in range(3):
        tickets.append(plan.moe_layer_host_submit(hx2[i & 1], dwr, dbias, dwg, dwu, dwd, hy2[i & 1]))
        if i:
            plan.moe_layer_host_wait(tickets[i - 1])
    plan.moe_layer_host_wait(tickets[-1])
    barrier()
    t0 = time.perf_counter()
    tickets = []
    for i in range(args.steps):
        tickets.append(plan.moe_layer_host_submit(hx2[i & 1], dwr, dbias, dwg, dwu, dwd, hy2[i & 1]))
        if i:
            plan.moe_layer_host_wait(tickets[i - 1])
    plan.moe_layer_host_wait(tickets[-1])
    ms_e2e = 1e3 * (time.perf_counter() - t0)
    torch.cuda.synchronize()
    code, detail = plan.moe_last_status()
    if code != 0:
        raise SystemExit(f"bench.py: device status {code} ({B.strerror(code)}), detail {detail}")

    ms_total, ms_e2e, ms_e2e_sync = max_over_ranks([ms_total, ms_e2e, ms_e2e_sync], "cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peak_kind = load_peaks()
    eb = w.elem_bytes
    rows = w.T * w.K
    ms_step = ms_total / args.steps
    value = whole_job_tokens_per_s(w.T, world, ms_step)

    # algorithmic work per launch of each stage
    disp_bytes = w.T * w.H * eb * (1 + w.K) + 12 * rows
    comb_bytes = w.T * w.H * eb * (w.K + 1) + 8 * rows
    route_bytes = w.T * w.H * eb + w.E * w.H * eb + 8 * rows
    gemm1_flops = 4.0 * rows * w.H * w.F
    gemm2_flops = 2.0 * rows * w.H * w.F
    sm = dict(zip(B.STAGES, stage_ms.tolist()))
    hbm_peak = peaks["hbm_gbs"]
    counts = plan.layer_tensor(3).cpu().numpy().astype(np.float64)
    routing_stats = {"hottest_expert_rows_over_T": float(counts.max() / w.T), "experts_without_rows": int((counts == 0).sum()),
                     "std_of_expert_share": float(np.std(counts / rows)), "tiles_used": int(np.sum((counts + 127) // 128)),
                     "tiles_if_dense": int((rows + 127) // 128)}
    stages = {
        "route": {"ms": sm["route"], "GBps": route_bytes / sm["route"] / 1e6 if sm["route"] > 0 else None},
        "dispatch": {"ms": sm["dispatch"], "GBps": disp_bytes / sm["dispatch"] / 1e6,
                     "frac_hbm": disp_bytes / sm["dispatch"] / 1e6 / hbm_peak,
                     "frac_hbm_nominal_8TBps": disp_bytes / sm["dispatch"] / 1e6 / 8000.0, "mode": dispatch},
        "combine": {"ms": sm["combine"], "GBps": comb_bytes / sm["combine"] / 1e6,
                    "frac_hbm": comb_bytes / sm["combine"] / 1e6 / hbm_peak,
                    "frac_hbm_nominal_8TBps": comb_bytes / sm["combine"] / 1e6 / 8000.0},
    }
    for name, nbytes in (("dispatch", disp_bytes), ("combine", comb_bytes)):
        us = plain_copy_us(nbytes) if rank == 0 else None
        if us:
            stages[name]["plain_copy_same_bytes_us"] = us
            stages[name]["time_vs_plain_copy"] = stages[name]["ms"] * 1e3 / us
    if w.identity_experts or w.dtype != inputs.BF16:
        dom = "dispatch"
        roofline = {"kernel": "dispatch", "bound": "hbm", "achieved": stages["dispatch"]["GBps"], "peak": hbm_peak,
                    "unit": "GB/s", "frac": stages["dispatch"]["frac_hbm"], "traffic": ncu_traffic_bytes(w.name),
                    "peak_source": f"{peak_kind} hbm_gbs"}
    else:
        t_ffn = sm["gemm1"] + sm["gemm2"]
        stages["ffn"] = {"ms": t_ffn, "TFLOPs": (gemm1_flops + gemm2_flops) / t_ffn / 1e9,
                         "launches": 2 if sm["gemm2"] > 0.02 * sm["gemm1"] else 1}
        if stages["ffn"]["launches"] == 2:
            stages["ffn_gemm1"] = {"ms": sm["gemm1"], "TFLOPs": gemm1_flops / sm["gemm1"] / 1e9}
            stages["ffn_gemm2"] = {"ms": sm["gemm2"], "TFLOPs": gemm2_flops / sm["gemm2"] / 1e9}
        ach = stages["ffn"]["TFLOPs"]
        # Algorithmic bytes of the two GEMMs: the weights of every expert that has rows, once; the rows in
        # and out; the intermediate written and read back.
        active = int((counts > 0).sum())
        ffn_bytes = 3.0 * active * w.F * w.H * eb + 2.0 * rows * w.H * eb + 2.0 * rows * w.F * eb
        stages["ffn"]["GBps"] = ffn_bytes / t_ffn / 1e6
        # Denominator: the burst cuBLAS figure when the timed region is shorter than a second (the part has not
        # settled under its power cap yet), the sustained one for longer runs; both fractions are reported.
        sustained = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
        long_run = ms_total >= 1000.0
        peak = sustained if long_run else peaks["bf16_tflops"]
        roofline = {"kernel": "ffn_tc_kernel (expert GEMM1 + SwiGLU + GEMM2, tcgen05)", "bound": "tensor",
                    "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak,
                    "traffic": ncu_traffic_bytes(w.name),
                    "peak_source": f"{peak_kind} " + ("bf16_tflops_sustained (timed region of %.1f s)" % (ms_total / 1e3) if long_run else
                                                      "bf16_tflops, the burst figure (timed region of %.0f ms)" % ms_total) +
                                   "; the kernel's clock is in clocks.ffn_kernel_sm_mhz",
                    "frac_of_burst_peak": ach / peaks["bf16_tflops"],
                    "frac_of_sustained_peak": ach / sustained,
                    "frac_of_nominal_2250": ach / 2250.0,
                    "useful_flops_per_launch": gemm1_flops + gemm2_flops}
        if ffn_bytes / (hbm_peak * 1e9) > (gemm1_flops + gemm2_flops) / (peaks["bf16_tflops"] * 1e12):
            # About a tile per expert: streaming the weights takes longer than the MMAs could, so the same
            # kernel is graded against the copy rate.
            roofline.update({"bound": "hbm", "achieved": stages["ffn"]["GBps"], "peak": hbm_peak, "unit": "GB/s",
                             "frac": stages["ffn"]["GBps"] / hbm_peak, "peak_source": f"{peak_kind} hbm_gbs",
                             "algorithmic_bytes_per_launch": ffn_bytes, "tensor_TFLOPs": ach})

    # the CPU oracle on a bounded sample of the same batch (N = 1 only)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        import oracle
        n = oracle_sample_tokens(w, oracle.num_threads())
        secs, threads = oracle_sample(w, n, x, wr, bias, wg, wu, wd)
        cpu = {"value": n / secs, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"first {n} of {w.T} tokens, whole layer, {secs:.1f} s"}

    if clocks.get("mean_power_w") and clocks.get("power_limit_w") and clocks["mean_power_w"] >= 0.93 * clocks["power_limit_w"]:
        roofline["power_note"] = ("the board ran at its power limit during the timed region (clocks.mean_power_w of "
                                  "clocks.power_limit_w): the kernel's clock, and with it both fractions, are set by the energy per step")
    h2d = w.T * w.H * eb
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == inputs.BF16 else "f32", "data": "synthetic",
            "config": workload_config(w, {"dispatch_mode": dispatch, "parallelism": f"replicas x{world}",
                                          "l2": "no flush: the per-step working set (weights + buffers, %.1f GB) "
                                                "exceeds the 126 MB L2" % ((3 * w.E * w.F * w.H * eb + 4 * rows * w.H * eb) / 1e9)}),
            "clocks": clocks, "gpu_launches": launches_per_step * args.steps,
            "e2e": {"value": whole_job_tokens_per_s(w.T, world, ms_e2e / args.steps), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": h2d,
                    "api": "moe_layer_host_submit/_wait: pinned host x and y, two steps in flight, host wall clock",
                    "one_step_at_a_time": whole_job_tokens_per_s(w.T, world, ms_e2e_sync / args.steps)},
            "roofline": roofline, "cpu_baseline": cpu, "stages": stages, "dominant": roofline["kernel"],
            "stages_from": "a separate pass with an event after every kernel and a synchronisation per step, run after the "
                           "timed steps: the stage times can add up to more than ms_per_step",
            "routing": routing_stats, "availability": availability}
    if overlap_arm is not None:
        line["availability_overlapped_launch"] = overlap_arm
    if world == 1 and args.also:
        # free the main workload's device memory first
        del plan, dx, dwr, dbias, dwg, dwu, dwd, y, wg, wu, wd
        torch.cuda.empty_cache()
        line["other_workloads"] = {WORKLOADS[name].name: brief_measurement(args, WORKLOADS[name]) for name in args.also.split(",")
                                   if name and WORKLOADS[name].name != w.name}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="c3", choices=sorted(WORKLOADS),
                    help="default: the largest full-layer configuration that fits one GPU (DeepSeek-V3-like)")
    ap.add_argument("--also", default=None,
                    help="comma-separated workloads measured briefly after the main one and reported under other_workloads "
                         "(default: c2 when the main workload is the default one)")
    ap.add_argument("--dispatch", default="auto", choices=["auto", "scan", "static", "paged", "ordered"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ffn-kernel", type=int, default=0, choices=[0, 1, 2],
                    help="0: tcgen05 one CTA per tile (default), 2: tcgen05 CTA pairs, 1: SIMT check path")
    ap.add_argument("--ffn-split", type=int, default=0, choices=[0, 1, 2],
                    help="expert GEMMs: 1 = one launch each, 2 = one launch for both, 0 = library default")
    ap.add_argument("--ffn-hot-min-tiles", type=int, default=0,
                    help="two-launch expert GEMMs: experts with at least this many tiles are walked as tensor-bound "
                         "work, interleaved with the weight-streaming-bound rest (0: library default, -1: off)")
    ap.add_argument("--route-filter", type=int, default=0, choices=[0, -1], help="-1: the router computes every expert's chain (no tensor-core filter)")
    ap.add_argument("--ffn-thin-tiles", type=int, default=0, help="-1: no transposed narrow form for small single tiles")
    ap.add_argument("--tp-shards", type=int, default=0,
                    help="expert + tensor parallelism: every expert cut into this many shards with a receive region each")
    ap.add_argument("--combine-mode", type=int, default=0, choices=[0, 1],
                    help="1: push-style combine (the expert kernel stores every result at its token's position)")
    ap.add_argument("--overlap", type=int, default=0,
                    help="with --dispatch ordered: dispatch inside the expert kernel's launch (1: half of the SMs dispatch, n: n CTAs)")
    args = ap.parse_args()
    if args.also is None:
        args.also = "c2" if args.workload == "c3" else ""
    w = WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_cuda(args, w)


if __name__ == "__main__":
    main()
