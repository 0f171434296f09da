"""Dispatch/combine-only sweep (identity experts): H = 7168, E = 256 on R = 32 logical ranks, top-8, bf16,
T from 128 to 65536 in powers of two, unbiased and Zipf(1.2) routing.  For every point it times the
dispatch stage (baseline scan scheme, the destination-agnostic paged scheme and the token-ordered
bulk-copy scheme) and the combine stage
with CUDA events and prints algorithmic GB/s and the fraction of the measured HBM copy bandwidth.

    python -m paper_2605_05888_b200.sweep [--max-t 65536] [--iters 20] [--markdown]
    python -m paper_2605_05888_b200.sweep --imbalance [--iters 20] [--markdown]

The second form is the imbalance study (Section VI-B of the paper varies the standard deviation of the
experts' load shares): the Mixtral-like layer (T 4096, H 4096, 8 experts, top-2, F 14336, bf16, real expert
GEMMs) with the router bias -s*ln(1+pi(e)) for s from 0 to 3; per point the measured standard deviation of
the experts' shares of the T*K rows, the hottest expert's share, the tiles used, and the layer time.

Algorithmic bytes: dispatch T*H*b*(1+K) + 12*T*K (row read once, written K times; indices in, slot and
source info out); combine T*H*b*(K+1) + 8*T*K.  Below T = 2048 the stages take a few microseconds and are
bound by launch latency, not bandwidth: read the microseconds there, not the GB/s.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

from . import binding as B
from . import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def hbm_peak_gbs() -> tuple[float, str]:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return json.load(open(path))["hbm_gbs"], "measured"
    return 6650.0, "fallback"


def time_point(w: inputs.Workload, mode: int, iters: int) -> dict:
    x = inputs.make_x(w)
    wr, bias = inputs.make_router(w)
    dx = torch.from_numpy(x).view(torch.int16).cuda().view(torch.bfloat16)
    dwr = torch.from_numpy(wr).view(torch.int16).cuda().view(torch.bfloat16)
    dbias = None if bias is None else torch.from_numpy(bias).cuda()
    plan = B.Plan(B.make_config(w.T, w.H, w.E, w.R, w.K, w.F, w.dtype, dispatch_mode=mode, identity_experts=1))
    y = torch.empty((w.T, w.H), dtype=torch.bfloat16, device="cuda")
    for _ in range(3):
        plan.moe_layer(dx, dwr, dbias, None, None, None, y)
    torch.cuda.synchronize()
    code, detail = plan.moe_last_status()
    assert code == 0, (code, detail)
    ms = np.array([plan.moe_layer_timed(dx, dwr, dbias, None, None, None, y) for _ in range(iters)])
    med = np.median(ms, axis=0)
    cnt = plan.layer_tensor(3).cpu().numpy()
    return {"dispatch_ms": float(med[B.STAGES.index("dispatch")]), "combine_ms": float(med[B.STAGES.index("combine")]),
            "route_ms": float(med[B.STAGES.index("route")]), "hottest_share": float(cnt.max() / w.T),
            "imbalance_std": float(np.std(cnt / (w.T * w.K)))}


def imbalance_point(w: inputs.Workload, weights, iters: int) -> dict:
    x = inputs.make_x(w)
    wr, bias = inputs.make_router(w)
    bf = lambda a: torch.from_numpy(a).view(torch.int16).cuda().view(torch.bfloat16)
    dx, dwr = bf(x), bf(wr)
    dbias = None if bias is None else torch.from_numpy(bias).cuda()
    plan = B.Plan(B.make_config(w.T, w.H, w.E, w.R, w.K, w.F, w.dtype))
    y = torch.empty((w.T, w.H), dtype=torch.bfloat16, device="cuda")
    for _ in range(5):
        plan.moe_layer(dx, dwr, dbias, *weights, y)
    torch.cuda.synchronize()
    code, detail = plan.moe_last_status()
    assert code == 0, (code, detail)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        plan.moe_layer(dx, dwr, dbias, *weights, y)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    cnt = plan.layer_tensor(3).cpu().numpy().astype(np.float64)
    rows = w.T * w.K
    return {"zipf_s": w.zipf_s, "std_of_expert_share": float(np.std(cnt / rows)), "hottest_share_of_rows": float(cnt.max() / rows),
            "tiles_used": int(np.sum((cnt + 127) // 128)), "tiles_if_dense": (rows + 127) // 128, "layer_ms": ms,
            "tokens_per_s": w.T / ms * 1e3}


def imbalance_sweep(iters: int, markdown: bool) -> None:
    base = inputs.C2
    wg, wu, wd = inputs.make_all_expert_weights(base)
    bf = lambda a: torch.from_numpy(a).view(torch.int16).cuda().view(torch.bfloat16)
    weights = (bf(wg), bf(wu), bf(wd))
    del wg, wu, wd
    rows = [imbalance_point(base.with_(zipf_s=s), weights, iters) for s in (0.0, 0.25, 0.5, 1.0, 1.5, 2.0, 3.0)]
    if not markdown:
        for r in rows:
            print(json.dumps(r))
        return
    print(f"Layer time = {iters} back-to-back `moe_layer` calls between two CUDA events, after 5 warm-ups.")
    print()
    print("| bias strength s | std of expert shares | hottest expert's share of rows | tiles used / dense | layer ms | tokens/s |")
    print("|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['zipf_s']:.2f} | {r['std_of_expert_share']:.4f} | {r['hottest_share_of_rows']:.3f} | {r['tiles_used']} / {r['tiles_if_dense']} | "
              f"{r['layer_ms']:.3f} | {r['tokens_per_s']:.3e} |")


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--min-t", type=int, default=128)
    ap.add_argument("--max-t", type=int, default=65536)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--markdown", action="store_true")
    ap.add_argument("--imbalance", action="store_true", help="the imbalance study on the Mixtral-like layer instead of the T sweep")
    args = ap.parse_args()
    if args.imbalance:
        imbalance_sweep(args.iters, args.markdown)
        return
    peak, kind = hbm_peak_gbs()
    rows = []
    T = args.min_t
    while T <= args.max_t:
        for zipf in (0.0, 1.2):
            w = inputs.C5(T, zipf)
            eb, n = w.elem_bytes, w.T * w.K
            disp_bytes = w.T * w.H * eb * (1 + w.K) + 12 * n
            comb_bytes = w.T * w.H * eb * (w.K + 1) + 8 * n
            scan = time_point(w, B.DISPATCH_SCAN, args.iters)
            paged = time_point(w, B.DISPATCH_ATOMIC_PAGED, args.iters)
            ordered = time_point(w, B.DISPATCH_ATOMIC_ORDERED, args.iters)
            rows.append({"T": T, "routing": "zipf1.2" if zipf else "uniform", "hottest_share": paged["hottest_share"],
                         "dispatch_scan_us": 1e3 * scan["dispatch_ms"], "dispatch_paged_us": 1e3 * paged["dispatch_ms"],
                         "dispatch_ordered_us": 1e3 * ordered["dispatch_ms"],
                         "dispatch_scan_GBps": disp_bytes / scan["dispatch_ms"] / 1e6,
                         "dispatch_paged_GBps": disp_bytes / paged["dispatch_ms"] / 1e6,
                         "dispatch_ordered_GBps": disp_bytes / ordered["dispatch_ms"] / 1e6,
                         "combine_us": 1e3 * paged["combine_ms"], "combine_GBps": comb_bytes / paged["combine_ms"] / 1e6})
            torch.cuda.empty_cache()
        T *= 2
    if args.markdown:
        print(f"HBM copy peak: {peak:.1f} GB/s ({kind}). Times are medians of {args.iters} runs, CUDA events around the stage.")
        print()
        print("| T | routing | hottest expert (rows/T) | dispatch scan us | GB/s | % | dispatch paged us | GB/s | % | dispatch ordered us | GB/s | % | combine us | GB/s | % |")
        print("|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|")
        for r in rows:
            print(f"| {r['T']} | {r['routing']} | {r['hottest_share']:.2f} | {r['dispatch_scan_us']:.1f} | "
                  f"{r['dispatch_scan_GBps']:.0f} | {100 * r['dispatch_scan_GBps'] / peak:.0f} | {r['dispatch_paged_us']:.1f} | "
                  f"{r['dispatch_paged_GBps']:.0f} | {100 * r['dispatch_paged_GBps'] / peak:.0f} | {r['dispatch_ordered_us']:.1f} | "
                  f"{r['dispatch_ordered_GBps']:.0f} | {100 * r['dispatch_ordered_GBps'] / peak:.0f} | {r['combine_us']:.1f} | "
                  f"{r['combine_GBps']:.0f} | {100 * r['combine_GBps'] / peak:.0f} |")
    else:
        for r in rows:
            print(json.dumps(r))


if __name__ == "__main__":
    main()
