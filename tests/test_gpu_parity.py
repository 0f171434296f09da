"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU oracle on
the same seeded inputs.  Routing indices and dispatch contents bit-exact (rows inside an expert
compared after sorting by source id: arrival order is free, Section IV-B of the paper), routing
weights within 1e-5 relative, combined output within 1e-4 (fp32, element-wise with an rms floor) /
2e-2 (bf16, per-token normwise) of the oracle: see parity_helpers.assert_output_close."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2605_05888_b200 import binding as B
from paper_2605_05888_b200 import inputs
import parity_helpers as Hh

pytestmark = pytest.mark.gpu
FP32, BF16 = inputs.FP32, inputs.BF16
MODES = [B.DISPATCH_SCAN, B.DISPATCH_ATOMIC_STATIC, B.DISPATCH_ATOMIC_PAGED, B.DISPATCH_ATOMIC_ORDERED]

SMALL = [
    inputs.C1,
    inputs.C1.with_(seed=1), inputs.C1.with_(seed=2),
    inputs.Workload("ragged_bf16", T=333, H=264, E=12, R=3, K=3, F=200, dtype=BF16),
    inputs.Workload("qwen_small", T=97, H=512, E=60, R=4, K=4, F=352, dtype=BF16),
    inputs.Workload("many_experts", T=300, H=256, E=256, R=32, K=8, F=128, dtype=BF16, zipf_s=1.0),
    inputs.Workload("k_equals_e", T=50, H=64, E=4, R=2, K=4, F=64, dtype=FP32),
    inputs.Workload("one_token", T=1, H=128, E=8, R=1, K=2, F=128, dtype=BF16),
    inputs.Workload("top1", T=130, H=128, E=16, R=4, K=1, F=136, dtype=BF16, zipf_s=1.2),
    # the limits of the entry points: K = 32 picks per token, with 64 and with 256 experts
    inputs.Workload("max_k", T=70, H=128, E=64, R=4, K=32, F=64, dtype=BF16),
    inputs.Workload("max_e_max_k", T=45, H=64, E=256, R=8, K=32, F=64, dtype=BF16, zipf_s=1.0),
]


def run_stages(w, mode, x, wr, bias, wg, wu, wd, ffn_kernel=0):
    plan = Hh.make_plan(w, mode, ffn_kernel=ffn_kernel)
    el = Hh.el_dtype(w)
    dx, dwr, dbias = Hh.to_dev(x), Hh.to_dev(wr), Hh.to_dev(bias)
    idx = torch.empty((w.T, w.K), dtype=torch.int32, device="cuda")
    tw = torch.empty((w.T, w.K), dtype=torch.float32, device="cuda")
    plan.moe_route(dx, dwr, dbias, idx, tw)
    rows = plan.P * 128
    recv = torch.zeros((rows, w.H), dtype=el, device="cuda")
    cnt = torch.empty(w.E, dtype=torch.int32, device="cuda")
    te = torch.empty(plan.P, dtype=torch.int32, device="cuda")
    src = torch.empty(rows, dtype=torch.int32, device="cuda")
    slot = torch.empty((w.T, w.K), dtype=torch.int32, device="cuda")
    plan.moe_dispatch(dx, idx, recv, cnt, te, src, slot)
    if w.identity_experts:
        out_rows = recv
    else:
        out_rows = torch.zeros((rows, w.H), dtype=el, device="cuda")
        plan.moe_expert_ffn(recv, te, Hh.to_dev(wg), Hh.to_dev(wu), Hh.to_dev(wd), out_rows)
    y = torch.empty((w.T, w.H), dtype=el, device="cuda")
    plan.moe_combine(out_rows, slot, tw, y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    return dict(plan=plan, idx=idx, tw=tw, recv=recv, cnt=cnt, te=te, src=src, slot=slot, out_rows=out_rows, y=y)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("w", SMALL, ids=lambda w: w.name + f"_s{w.seed}")
def test_stages_match_oracle(w, mode):
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)
    g = run_stages(w, mode, x, wr, bias, wg, wu, wd)
    Hh.check_route(g["idx"], g["tw"], ref["topk_idx"], ref["topk_w"])
    Hh.check_dispatch(w, g["plan"].P, x, ref["topk_idx"], ref, g["recv"], g["cnt"], g["te"], g["src"], g["slot"])
    # expert outputs row by row (canonical order) and the combined result
    slot = g["slot"].cpu().numpy()
    got_rows = Hh.to_host_f64(g["out_rows"])[slot.ravel()]
    ref_rows = ref["out_rows"][ref["slot_of"].ravel()]
    Hh.assert_output_close(got_rows, ref_rows, w.dtype, "expert outputs")
    Hh.assert_output_close(Hh.to_host_f64(g["y"]), ref["y"], w.dtype, "combined output")
    if w.dtype == BF16:   # and within a bf16 step of the restatement that rounds where the kernels store bf16
        stored = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd, bf16_storage=True)
        Hh.assert_close_to_bf16_storage(Hh.to_host_f64(g["y"]), stored, "combined output")


@pytest.mark.parametrize("w", [SMALL[3], SMALL[4], SMALL[5]], ids=lambda w: w.name)
def test_simt_ffn_matches_oracle_bf16(w):
    """The fp32-FMA expert kernel on bf16 data: the second device implementation of step 3."""
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)
    g = run_stages(w, B.DISPATCH_SCAN, x, wr, bias, wg, wu, wd, ffn_kernel=1)
    Hh.assert_output_close(Hh.to_host_f64(g["y"]), ref["y"], w.dtype)


@pytest.mark.parametrize("split", [1, 2])
@pytest.mark.parametrize("w", [SMALL[3], SMALL[4], SMALL[5], SMALL[7],
                               inputs.Workload("three_tiles", T=700, H=320, E=4, R=2, K=2, F=392, dtype=BF16)],
                         ids=lambda w: w.name)
@pytest.mark.parametrize("kernel", [0, 2])
def test_tensor_core_ffn_forms_match_oracle(w, split, kernel):
    """Both forms of the tensor-core expert kernel - one CTA per tile (0) and the cta_group::2 form (2: two
    tiles of an expert per MMA; experts with an odd number of tiles leave one CTA of the last pair without
    work) - each as one launch for both GEMMs (per-tile counters gate GEMM2) and as two launches."""
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_PAGED, ffn_kernel=kernel, ffn_split=split)
    y = torch.empty((w.T, w.H), dtype=Hh.el_dtype(w), device="cuda")
    plan.moe_layer(Hh.to_dev(x), Hh.to_dev(wr), Hh.to_dev(bias), Hh.to_dev(wg), Hh.to_dev(wu), Hh.to_dev(wd), y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    Hh.assert_output_close(Hh.to_host_f64(y), ref["y"], w.dtype)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("w", [inputs.C1, SMALL[3], SMALL[5], SMALL[9], SMALL[10], inputs.C5(512), inputs.C5(256, 1.2)],
                         ids=lambda w: w.name)
def test_fused_layer_matches_oracle(w, mode):
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)
    plan = Hh.make_plan(w, mode)
    y = torch.empty((w.T, w.H), dtype=Hh.el_dtype(w), device="cuda")
    plan.moe_layer(Hh.to_dev(x), Hh.to_dev(wr), Hh.to_dev(bias), Hh.to_dev(wg), Hh.to_dev(wu), Hh.to_dev(wd), y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    assert plan.moe_last_launch_count() >= 3
    Hh.check_route(plan.layer_tensor(0), plan.layer_tensor(1), ref["topk_idx"], ref["topk_w"])
    Hh.check_dispatch(w, plan.P, x, ref["topk_idx"], ref, plan.layer_tensor(2), plan.layer_tensor(3),
                      plan.layer_tensor(4), plan.layer_tensor(5), plan.layer_tensor(6))
    Hh.assert_output_close(Hh.to_host_f64(y), ref["y"], w.dtype)
    # host-buffer entry point gives the same bytes
    hx = torch.from_numpy(x.view(np.int16) if x.dtype == np.uint16 else x).pin_memory()
    hy = torch.empty_like(hx).pin_memory()
    plan.moe_layer_host(hx, Hh.to_dev(wr), Hh.to_dev(bias), Hh.to_dev(wg), Hh.to_dev(wu), Hh.to_dev(wd), hy)
    y_bits = Hh.to_host_bits(y)
    assert np.array_equal(hy.numpy().view(y_bits.dtype), y_bits)


def test_identity_experts_closed_form():
    """Identity experts make the layer return x * sum_k w (a property that holds at any size)."""
    w = inputs.C5(2048, 1.2)
    x, wr, bias, *_ = Hh.oracle_inputs(w, with_experts=False)
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_PAGED)
    y = torch.empty((w.T, w.H), dtype=torch.bfloat16, device="cuda")
    dx = Hh.to_dev(x)
    plan.moe_layer(dx, Hh.to_dev(wr), Hh.to_dev(bias), None, None, None, y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    ws = plan.layer_tensor(1).double().sum(1, keepdim=True)
    ref = (dx.double() * ws).cpu().numpy()
    Hh.assert_output_close(Hh.to_host_f64(y), ref, w.dtype)


# ------------------------------------------------------------------ router edge cases
def test_router_tie_patterns_exhaustive():
    """H = 8 >= E and Wr = [I | 0] make the logits equal x[:, :E]; x runs over {-1,0,1}^E, every tie
    pattern of the top-K selection, K = 1..E."""
    for E in (2, 3, 5):
        grid = np.array(list(itertools.product([-1.0, 0.0, 1.0], repeat=E)), np.float32)
        T = grid.shape[0]
        x = np.zeros((T, 8), np.float32)
        x[:, :E] = grid
        wr = np.zeros((E, 8), np.float32)
        wr[np.arange(E), np.arange(E)] = 1.0
        for K in range(1, E + 1):
            w = inputs.Workload("ties", T=T, H=8, E=E, R=1, K=K, F=8, dtype=FP32)
            plan = Hh.make_plan(w, B.DISPATCH_SCAN)
            idx = torch.empty((T, K), dtype=torch.int32, device="cuda")
            tw = torch.empty((T, K), dtype=torch.float32, device="cuda")
            plan.moe_route(Hh.to_dev(x), Hh.to_dev(wr), None, idx, tw)
            ridx, rw, _ = oracle.route(x, wr, None, K, FP32)
            Hh.check_route(idx, tw, ridx, rw)


@pytest.mark.parametrize("E", [60, 160])   # the narrow router; the tensor-core filter of the wide one
@pytest.mark.parametrize("renorm", [0, 1])
def test_router_renormalize_and_bias(renorm, E):
    w = inputs.Workload("renorm", T=200, H=512, E=E, R=4, K=4, F=8, dtype=BF16, zipf_s=1.0, seed=3)
    x, wr, bias, *_ = Hh.oracle_inputs(w, with_experts=False)
    cfg = B.make_config(w.T, w.H, w.E, w.R, w.K, w.F, w.dtype, renormalize=renorm)
    plan = B.Plan(cfg)
    idx = torch.empty((w.T, w.K), dtype=torch.int32, device="cuda")
    tw = torch.empty((w.T, w.K), dtype=torch.float32, device="cuda")
    plan.moe_route(Hh.to_dev(x), Hh.to_dev(wr), Hh.to_dev(bias), idx, tw)
    ridx, rw, _ = oracle.route(x, wr, bias, w.K, w.dtype, renormalize=renorm)
    Hh.check_route(idx, tw, ridx, rw)


# Every shape of the two router kernels: the narrow kernel's four lane layouts (E <= 8, 16, 32, 64), each
# with a block boundary inside T and an h range that ends inside a chunk, in both dtypes; the wide kernel
# with every register-tile height it picks (4 to 8 tokens per thread follows from T on a 148-SM part:
# T <= 4736 -> 4, <= 5920 -> 5, <= 7104 -> 6, <= 8288 -> 7, <= 9472 -> 8) and E below and at 256.
ROUTER_SHAPES = [
    # (T, H, E, K, dtype, zipf_s)
    (77, 264, 7, 2, BF16, 0.0), (1100, 520, 8, 3, BF16, 1.0), (45, 132, 5, 5, FP32, 0.0),
    (333, 1032, 16, 2, BF16, 0.0), (90, 260, 13, 4, FP32, 1.0),
    (70, 520, 32, 6, BF16, 0.0), (1500, 264, 24, 2, BF16, 1.0), (33, 68, 17, 3, FP32, 0.0),
    (130, 776, 60, 4, BF16, 0.0), (1030, 136, 64, 8, BF16, 1.0), (21, 132, 33, 2, FP32, 0.0),
    (200, 72, 65, 8, BF16, 0.0), (4000, 40, 256, 8, BF16, 1.0), (5000, 40, 200, 4, BF16, 0.0),
    (6500, 40, 256, 8, BF16, 1.0), (8000, 40, 129, 2, BF16, 0.0), (9000, 40, 256, 8, BF16, 1.0),
    (300, 36, 100, 5, FP32, 1.0), (5100, 20, 256, 3, FP32, 0.0),
]


@pytest.mark.parametrize("shape", ROUTER_SHAPES, ids=lambda s: f"T{s[0]}_H{s[1]}_E{s[2]}_K{s[3]}_d{s[4]}_z{s[5]}")
def test_router_every_kernel_shape(shape):
    T, H, E, K, dtype, zipf = shape
    w = inputs.Workload("router_shape", T=T, H=H, E=E, R=1, K=K, F=8, dtype=dtype, zipf_s=zipf, seed=11,
                        identity_experts=True)
    x, wr, bias, *_ = Hh.oracle_inputs(w, with_experts=False)
    ridx, rw, _ = oracle.route(x, wr, bias, K, dtype)
    for route_filter in ((0, -1) if (dtype == BF16 and E > 64) else (0,)):   # -1: the all-chains kernel for many experts
        plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_PAGED, route_filter=route_filter)
        idx = torch.empty((T, K), dtype=torch.int32, device="cuda")
        tw = torch.empty((T, K), dtype=torch.float32, device="cuda")
        plan.moe_route(Hh.to_dev(x), Hh.to_dev(wr), Hh.to_dev(bias), idx, tw)
        torch.cuda.synchronize()
        Hh.check_route(idx, tw, ridx, rw)


# ------------------------------------------------------------------ dispatch edge cases
@pytest.mark.parametrize("mode", MODES)
def test_dispatch_all_tokens_to_one_expert_and_empty_experts(mode):
    w = inputs.Workload("skew", T=700, H=64, E=8, R=2, K=2, F=8, dtype=BF16)
    x = inputs.make_x(w)
    idx = np.zeros((w.T, w.K), np.int32)
    idx[:, 0], idx[:, 1] = 5, 2           # experts 5 and 2 get T rows each, the others none
    ref = oracle.dispatch(x, idx, w.E, w.R, w.dtype)
    plan = Hh.make_plan(w, mode)
    rows = plan.P * 128
    recv = torch.zeros((rows, w.H), dtype=torch.bfloat16, device="cuda")
    cnt = torch.empty(w.E, dtype=torch.int32, device="cuda")
    te = torch.empty(plan.P, dtype=torch.int32, device="cuda")
    src = torch.empty(rows, dtype=torch.int32, device="cuda")
    slot = torch.empty((w.T, w.K), dtype=torch.int32, device="cuda")
    plan.moe_dispatch(Hh.to_dev(x), Hh.to_dev(idx), recv, cnt, te, src, slot)
    assert plan.moe_last_status() == (0, 0)
    Hh.check_dispatch(w, plan.P, x, idx, ref, recv, cnt, te, src, slot)


def test_static_region_overflow_is_reported_not_silent():
    """Mode 1 with regions smaller than the load: the status word says overflow and names an expert,
    counts stay exact, dropped assignments get slot -1, nothing is written out of bounds."""
    w = inputs.Workload("overflow", T=600, H=64, E=4, R=1, K=1, F=8, dtype=BF16)
    x = inputs.make_x(w)
    idx = np.full((w.T, 1), 3, np.int32)
    cfg = B.make_config(w.T, w.H, w.E, w.R, w.K, w.F, w.dtype, dispatch_mode=B.DISPATCH_ATOMIC_STATIC,
                        capacity_rows=256)
    plan = B.Plan(cfg)
    rows = plan.P * 128
    guard = torch.full((rows + 128, w.H), 7.0, dtype=torch.bfloat16, device="cuda")
    cnt = torch.empty(w.E, dtype=torch.int32, device="cuda")
    te = torch.empty(plan.P, dtype=torch.int32, device="cuda")
    src = torch.empty(rows, dtype=torch.int32, device="cuda")
    slot = torch.empty((w.T, w.K), dtype=torch.int32, device="cuda")
    plan.moe_dispatch(Hh.to_dev(x), Hh.to_dev(idx), guard[:rows], cnt, te, src, slot)
    code, detail = plan.moe_last_status()
    assert code == -5 and detail == 3
    assert cnt.cpu().tolist() == [0, 0, 0, 600]
    s = slot.cpu().numpy().ravel()
    assert (s >= 0).sum() == 256 and (s == -1).sum() == 600 - 256
    assert torch.all(guard[rows:] == 7.0)


def test_bad_arguments_are_refused_on_the_host():
    cfg = B.make_config(16, 100, 8, 2, 2, 64, BF16)      # H*2 bytes not a multiple of 16
    with pytest.raises(B.MoeError) as ei:
        B.moe_workspace_bytes(cfg)
    assert ei.value.code == -2
    with pytest.raises(B.MoeError):
        B.moe_workspace_bytes(B.make_config(16, 128, 8, 3, 2, 64, BF16))   # E % R != 0
    with pytest.raises(B.MoeError):
        B.moe_workspace_bytes(B.make_config(16, 128, 8, 2, 9, 64, BF16))   # K > E


# ------------------------------------------------------------------ availability counters and the bounded wait
def _dispatch_with_counters(w, plan, dx, didx):
    rows = plan.P * 128
    b = dict(recv=torch.zeros((rows, w.H), dtype=Hh.el_dtype(w), device="cuda"),
             cnt=torch.empty(w.E, dtype=torch.int32, device="cuda"), te=torch.empty(plan.P, dtype=torch.int32, device="cuda"),
             src=torch.empty(rows, dtype=torch.int32, device="cuda"),
             slot=torch.empty((w.T, w.K), dtype=torch.int32, device="cuda"),
             tile_count=torch.full((plan.P,), 77, dtype=torch.int32, device="cuda"),
             rows_done=torch.full((1,), 77, dtype=torch.int32, device="cuda"))
    plan.moe_dispatch(dx, didx, b["recv"], b["cnt"], b["te"], b["src"], b["slot"], b["tile_count"], b["rows_done"])
    return b


@pytest.mark.parametrize("mode", MODES)
def test_dispatch_availability_counters_and_gated_consumer(mode):
    """Section IV-D in software: after dispatch every tile's status counter equals the rows stored in it
    and the global counter equals T*K; the tensor-core consumer gated on those counters gives the same
    result as the ungated one."""
    w = SMALL[3]
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)
    plan = Hh.make_plan(w, mode)
    dx = Hh.to_dev(x)
    b = _dispatch_with_counters(w, plan, dx, Hh.to_dev(ref["topk_idx"]))
    torch.cuda.synchronize()
    assert int(b["rows_done"][0]) == w.T * w.K
    per_tile = torch.bincount(b["slot"].flatten().long() // 128, minlength=plan.P).int()
    assert torch.equal(b["tile_count"], per_tile)
    out = torch.zeros_like(b["recv"])
    plan.moe_expert_ffn(b["recv"], b["te"], Hh.to_dev(wg), Hh.to_dev(wu), Hh.to_dev(wd), out, b["tile_count"], b["rows_done"])
    y = torch.empty((w.T, w.H), dtype=Hh.el_dtype(w), device="cuda")
    plan.moe_combine(out, b["slot"], Hh.to_dev(ref["topk_w"]), y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    Hh.assert_output_close(Hh.to_host_f64(y), ref["y"], w.dtype)


@pytest.mark.parametrize("mode", MODES)
def test_availability_trace_orders_the_events(mode):
    """With the trace on, every tile that holds 128 rows has a ready time between the dispatch start and
    the all-ready time, tiles with fewer rows have none, and the layer's result is unchanged."""
    w = inputs.Workload("trace", T=900, H=264, E=12, R=3, K=3, F=136, dtype=BF16, zipf_s=1.0, seed=9)
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    args = [Hh.to_dev(a) for a in (x, wr, bias, wg, wu, wd)]
    plan = Hh.make_plan(w, mode)
    y0 = torch.empty((w.T, w.H), dtype=Hh.el_dtype(w), device="cuda")
    plan.moe_layer(*args, y0)
    plan.moe_availability_trace(True)
    y1 = torch.empty_like(y0)
    plan.moe_layer(*args, y1)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    tr = plan.layer_tensor(8).cpu().numpy()
    cnt = plan.layer_tensor(3).cpu().numpy()
    te = plan.layer_tensor(4).cpu().numpy()
    slot = plan.layer_tensor(6).cpu().numpy()
    per_tile = np.bincount(slot.ravel() // 128, minlength=plan.P)
    t0, t_all, ready = tr[0], tr[1], tr[2:]
    assert t0 > 0 and t_all >= t0
    full = per_tile == 128
    assert full.any() and (~full & (te >= 0)).any()
    assert (ready[full] >= t0).all() and (ready[full] <= t_all).all()
    assert (ready[~full] == 0).all()
    assert cnt.sum() == w.T * w.K
    assert torch.equal(y0, y1)
    plan.moe_availability_trace(False)


@pytest.mark.parametrize("kernel", [0, 2])
@pytest.mark.parametrize("split", [1, 2])
def test_expert_kernel_can_be_called_again_without_a_dispatch_in_between(split, kernel):
    """The expert kernel hands its items out through device counters and gates GEMM2 on per-tile GEMM1
    counters; it puts all of them back to zero itself.  Three calls in a row on one dispatch result (the
    counter-gated form, where no dispatch resets anything in between), each with DIFFERENT expert weights:
    a GEMM2 item that trusted the previous call's counters would read the previous call's intermediate,
    so every call is checked against the oracle for its own weights."""
    w = inputs.Workload("many_items", T=700, H=520, E=12, R=3, K=3, F=1032, dtype=BF16, seed=5)  # 288 items for 148 CTAs
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_PAGED, ffn_split=split, ffn_kernel=kernel)
    dx = Hh.to_dev(x)
    b = _dispatch_with_counters(w, plan, dx, Hh.to_dev(ref["topk_idx"]))
    outs = []
    for call in range(3):
        cwg, cwu, cwd = inputs.make_all_expert_weights(w.with_(seed=5 + 17 * call))
        out = torch.zeros_like(b["recv"])
        plan.moe_expert_ffn(b["recv"], b["te"], Hh.to_dev(cwg), Hh.to_dev(cwu), Hh.to_dev(cwd), out, b["tile_count"],
                            b["rows_done"])
        outs.append((out, cwg, cwu, cwd))
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    for out, cwg, cwu, cwd in outs:
        y = torch.empty((w.T, w.H), dtype=Hh.el_dtype(w), device="cuda")
        plan.moe_combine(out, b["slot"], Hh.to_dev(ref["topk_w"]), y)
        torch.cuda.synchronize()
        want = Hh.oracle_layer_for(w, x, wr, bias, cwg, cwu, cwd)
        Hh.assert_output_close(Hh.to_host_f64(y), want["y"], w.dtype)


@pytest.mark.parametrize("mode", MODES)
def test_expert_id_outside_the_range_is_reported_and_dropped(mode):
    """A caller-supplied topk_idx with an id that is no expert: the status word says bad argument and names
    the token, the assignment gets slot -1 and no row, every other assignment is dispatched as usual, and
    nothing outside the buffers is written (guard rows stay intact)."""
    w = inputs.Workload("bad_id", T=200, H=64, E=8, R=2, K=2, F=8, dtype=BF16)
    x = inputs.make_x(w)
    rng = np.random.default_rng(4)
    idx = np.stack([rng.permutation(w.E)[:w.K] for _ in range(w.T)]).astype(np.int32)
    idx[77, 1] = w.E + 5
    plan = Hh.make_plan(w, mode)
    rows = plan.P * 128
    guard = torch.full((rows + 128, w.H), 7.0, dtype=torch.bfloat16, device="cuda")
    cnt = torch.empty(w.E, dtype=torch.int32, device="cuda")
    te = torch.empty(plan.P, dtype=torch.int32, device="cuda")
    src = torch.empty(rows, dtype=torch.int32, device="cuda")
    slot = torch.empty((w.T, w.K), dtype=torch.int32, device="cuda")
    plan.moe_dispatch(Hh.to_dev(x), Hh.to_dev(idx), guard[:rows], cnt, te, src, slot)
    assert plan.moe_last_status() == (-1, 77)
    s = slot.cpu().numpy()
    assert s[77, 1] == -1 and (s.ravel() >= 0).sum() == w.T * w.K - 1
    good = idx.ravel() < w.E
    assert np.array_equal(cnt.cpu().numpy(), np.bincount(idx.ravel()[good], minlength=w.E))
    recv_h = Hh.to_host_bits(guard[:rows])
    flat = s.ravel()
    assert recv_h[flat[good]].tobytes() == np.repeat(x, w.K, axis=0)[good].tobytes()
    assert torch.all(guard[rows:] == 7.0)


@pytest.mark.parametrize("kernel", [0, 2])
def test_consumer_wait_runs_out_and_reports_it(kernel):
    """A flag that nothing sets: the consumer is given availability counters that stay at zero.  Its
    bounded wait (50 ms here) runs out, the kernel returns on its own, the status word says timeout
    and names the wait, and the same plan then runs a correct layer: nothing hangs, the context lives."""
    w = SMALL[3]
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_PAGED, ffn_kernel=kernel, wait_limit_ns=50_000_000)
    dx, dwg, dwu, dwd = Hh.to_dev(x), Hh.to_dev(wg), Hh.to_dev(wu), Hh.to_dev(wd)
    b = _dispatch_with_counters(w, plan, dx, Hh.to_dev(ref["topk_idx"]))
    never = torch.zeros(plan.P + 1, dtype=torch.int32, device="cuda")
    out = torch.zeros_like(b["recv"])
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    plan.moe_expert_ffn(b["recv"], b["te"], dwg, dwu, dwd, out, never[:plan.P], never[plan.P:])
    t1.record()
    code, detail = plan.moe_last_status()
    # MOE_ERR_TIMEOUT; the wait site is the producer's tile-availability wait (7) or, since every role's wait
    # has the same bound, the MMA (4) or epilogue (5) wait that starved behind it: the first to expire is kept
    assert code == -6 and detail in (7, 4, 5, 8), (code, detail)
    assert t0.elapsed_time(t1) < 2000.0
    y = torch.empty((w.T, w.H), dtype=Hh.el_dtype(w), device="cuda")
    plan.moe_layer(dx, Hh.to_dev(wr), Hh.to_dev(bias), dwg, dwu, dwd, y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    Hh.assert_output_close(Hh.to_host_f64(y), ref["y"], w.dtype)


# ------------------------------------------------------------------ dispatch and experts in one launch
OVERLAP_CASES = [SMALL[3], SMALL[4], SMALL[5], SMALL[7],
                 inputs.Workload("three_tiles", T=700, H=320, E=4, R=2, K=2, F=392, dtype=BF16),
                 inputs.Workload("many_items", T=2100, H=520, E=12, R=3, K=3, F=1032, dtype=BF16, seed=5, zipf_s=1.0),
                 inputs.Workload("long_rows", T=260, H=9216, E=8, R=2, K=2, F=128, dtype=BF16),
                 inputs.Workload("max_k_overlapped", T=70, H=128, E=64, R=4, K=32, F=64, dtype=BF16)]   # rows of 18 KB: two chunks per row


@pytest.mark.parametrize("split", [1, 2])
@pytest.mark.parametrize("w", OVERLAP_CASES, ids=lambda w: w.name)
def test_overlapped_dispatch_and_experts_match_oracle(w, split):
    """Section IV-D end to end: the launch that computes the experts also dispatches (its first CTAs walk the
    tokens in ascending order and raise the tiles' status counters, the others start on a tile when its counter
    reaches the rows the tile will hold).  Routing, dispatch contents and output against the oracle; both as one
    launch for the two GEMMs and as two."""
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_ORDERED, overlap=1, ffn_split=split)
    y = torch.empty((w.T, w.H), dtype=Hh.el_dtype(w), device="cuda")
    args = [Hh.to_dev(a) for a in (x, wr, bias, wg, wu, wd)]
    for _ in range(2):      # twice: the second call meets the counters as the first one left them
        # a row that a consumer read before its producer had stored it would show: the pool holds 1e30 everywhere
        plan.layer_tensor(2).fill_(1.0e30)
        plan.moe_layer(*args, y)
        torch.cuda.synchronize()
        assert plan.moe_last_status() == (0, 0)
        router = 2 if (w.dtype == BF16 and w.E > 64) else 1                     # many experts on bf16: filter + refine
        assert plan.moe_last_launch_count() == router + 1 + (2 if split == 1 else 1)   # router, expert launch(es) carrying the dispatch, combine
        Hh.check_route(plan.layer_tensor(0), plan.layer_tensor(1), ref["topk_idx"], ref["topk_w"])
        Hh.check_dispatch(w, plan.P, x, ref["topk_idx"], ref, plan.layer_tensor(2), plan.layer_tensor(3),
                          plan.layer_tensor(4), plan.layer_tensor(5), plan.layer_tensor(6))
        Hh.assert_output_close(Hh.to_host_f64(y), ref["y"], w.dtype)
    # the same bytes as the stream-ordered launches give
    plan2 = Hh.make_plan(w, B.DISPATCH_ATOMIC_ORDERED, ffn_split=split)
    y2 = torch.empty_like(y)
    plan2.moe_layer(*args, y2)
    torch.cuda.synchronize()
    assert torch.equal(y, y2)


def test_overlapped_consumer_wait_runs_out_and_reports_it():
    """The consumer's wait for a tile's status counter, in the overlapped launch, with a limit far below the time
    the producers need (1 microsecond): waits run out, the kernel returns by itself with MOE_ERR_TIMEOUT and a
    wait site, nothing hangs, and a plan with the normal limit then computes the right layer."""
    w = inputs.Workload("overlap_timeout", T=4096, H=2048, E=8, R=2, K=2, F=256, dtype=BF16)
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    args = [Hh.to_dev(a) for a in (x, wr, bias, wg, wu, wd)]
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_ORDERED, overlap=1, wait_limit_ns=1000)
    y = torch.empty((w.T, w.H), dtype=torch.bfloat16, device="cuda")
    # The dispatch gives up half-way too (its own waits have the same limit) and leaves entries of slot_of and of
    # the source information unwritten: whatever they hold must not be used as a row number by the later stages.
    plan.layer_tensor(6).fill_(2 ** 31 - 1)
    plan.layer_tensor(5).fill_(2 ** 31 - 1)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    plan.moe_layer(*args, y)
    t1.record()
    code, detail = plan.moe_last_status()
    assert code == -6 and detail in (3, 4, 5, 7, 8), (code, detail)
    assert t0.elapsed_time(t1) < 2000.0
    good = Hh.make_plan(w, B.DISPATCH_ATOMIC_ORDERED, overlap=1)
    good.moe_layer(*args, y)
    torch.cuda.synchronize()
    assert good.moe_last_status() == (0, 0)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)
    Hh.assert_output_close(Hh.to_host_f64(y), ref["y"], w.dtype)


def test_overlapped_launch_starts_expert_work_before_the_dispatch_ends():
    """The timeline of one traced overlapped layer: full tiles appear throughout the dispatch (ascending token
    order: the first one early), and the first GEMM1 item begins to load before the last row has been stored."""
    w = inputs.Workload("overlap_trace", T=8192, H=2048, E=8, R=2, K=2, F=512, dtype=BF16)
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    args = [Hh.to_dev(a) for a in (x, wr, bias, wg, wu, wd)]
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_ORDERED, overlap=1)
    y = torch.empty((w.T, w.H), dtype=torch.bfloat16, device="cuda")
    plan.moe_layer(*args, y)
    plan.moe_availability_trace(True)
    plan.layer_tensor(9).zero_()
    plan.moe_layer(*args, y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    tr = plan.layer_tensor(8).cpu().numpy()
    items = plan.layer_tensor(9).cpu().numpy()
    t0, t_all, ready = tr[0], tr[1], tr[2:]
    full = ready[ready > 0]
    assert full.size > 0 and t_all > t0
    first_tile = (full.min() - t0) / (t_all - t0)
    started = items[items[:, 0] > 0]
    gemm1 = started[(started[:, 2] & 1) == 0]
    assert gemm1[:, 0].min() < t_all, "no expert item began before the dispatch was over"
    assert first_tile < 0.5, f"first full tile only after {first_tile:.2f} of the dispatch"
    plan.moe_availability_trace(False)


# ------------------------------------------------------------------ push-style combine
PUSH_CASES = [SMALL[3], SMALL[4], SMALL[5], SMALL[7], SMALL[8],
              inputs.Workload("three_tiles", T=700, H=320, E=4, R=2, K=2, F=392, dtype=BF16),
              inputs.Workload("half_tiles", T=900, H=264, E=6, R=3, K=2, F=136, dtype=BF16, zipf_s=1.0, seed=2)]


@pytest.mark.parametrize("w", PUSH_CASES, ids=lambda w: w.name)
def test_push_combine_stages_match_oracle_and_the_gather_path(w):
    """Section IV-B, all-to-all combine: the expert kernel reads the source information of every row after its
    final GEMM and stores the result at the token's position t*K+k; the reduction then reads K consecutive rows.
    Through the C ABI (moe_expert_ffn_push, moe_combine_staged): every staged row is the expert output of its
    assignment, y matches the oracle, and y is the same bytes as the gather path's."""
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)
    g = run_stages(w, B.DISPATCH_ATOMIC_PAGED, x, wr, bias, wg, wu, wd)          # the gather path, for comparison
    plan = g["plan"]
    staged = torch.full((w.T * w.K, w.H), 7.0, dtype=torch.bfloat16, device="cuda")
    plan.moe_expert_ffn_push(g["recv"], g["te"], g["src"], Hh.to_dev(wg), Hh.to_dev(wu), Hh.to_dev(wd), staged)
    y = torch.empty((w.T, w.H), dtype=torch.bfloat16, device="cuda")
    plan.moe_combine_staged(staged, g["slot"], g["tw"], y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    slot = g["slot"].flatten().long()
    assert torch.equal(staged, g["out_rows"][slot]), "a staged row is not the expert output of its assignment"
    assert torch.equal(y, g["y"])
    Hh.assert_output_close(Hh.to_host_f64(y), ref["y"], w.dtype)


@pytest.mark.parametrize("overlap", [0, 1])
@pytest.mark.parametrize("mode", [B.DISPATCH_SCAN, B.DISPATCH_ATOMIC_PAGED, B.DISPATCH_ATOMIC_ORDERED])
@pytest.mark.parametrize("w", [SMALL[3], SMALL[4], SMALL[5]], ids=lambda w: w.name)
def test_layer_with_push_combine(w, mode, overlap):
    if overlap and mode != B.DISPATCH_ATOMIC_ORDERED:
        pytest.skip("the overlapped launch belongs to the ordered dispatch")
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)
    args = [Hh.to_dev(a) for a in (x, wr, bias, wg, wu, wd)]
    plan = Hh.make_plan(w, mode, combine_mode=1, overlap=overlap)
    y = torch.empty((w.T, w.H), dtype=torch.bfloat16, device="cuda")
    plan.moe_layer(*args, y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    Hh.assert_output_close(Hh.to_host_f64(y), ref["y"], w.dtype)
    gather = Hh.make_plan(w, mode)
    y2 = torch.empty_like(y)
    gather.moe_layer(*args, y2)
    torch.cuda.synchronize()
    assert torch.equal(y, y2)


def test_push_combine_is_refused_where_it_is_not_built():
    with pytest.raises(B.MoeError) as ei:
        B.moe_workspace_bytes(B.make_config(64, 128, 8, 2, 2, 64, FP32, combine_mode=1))
    assert ei.value.code == -3


# ------------------------------------------------------------------ expert + tensor parallelism
TP_CASES = [(inputs.Workload("tp_bf16", T=333, H=264, E=12, R=3, K=3, F=400, dtype=BF16), 2),
            (inputs.Workload("tp_bf16_4", T=700, H=320, E=4, R=2, K=2, F=1024, dtype=BF16, zipf_s=1.0), 4),
            (inputs.Workload("tp_many", T=300, H=256, E=64, R=8, K=8, F=256, dtype=BF16, zipf_s=1.0), 4),
            (inputs.Workload("tp_filtered_router", T=260, H=512, E=128, R=8, K=4, F=256, dtype=BF16, zipf_s=1.0), 2),  # 128 experts: the router's filter path
            (inputs.Workload("tp_fp32", T=130, H=128, E=8, R=2, K=2, F=192, dtype=FP32), 3)]


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("case", TP_CASES, ids=lambda c: f"{c[0].name}_S{c[1]}")
def test_tp_shards_layer_matches_oracle(case, mode):
    """Section VII: one receive region per TP shard, every row stored to each.  Routing (every pick listed once per
    shard), dispatch contents of the E*S regions and the output against the oracle's TP layer - which itself equals
    the plain layer - in every dispatch scheme; the output also agrees with the same plan without shards."""
    w, S = case
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd, tp_shards=S)
    args = [Hh.to_dev(a) for a in (x, wr, bias, wg, wu, wd)]
    plan = Hh.make_plan(w, mode, tp_shards=S)
    assert plan.P == (w.T * w.K * S // 128 + w.E * S if mode != B.DISPATCH_ATOMIC_STATIC else plan.P)
    y = torch.empty((w.T, w.H), dtype=Hh.el_dtype(w), device="cuda")
    plan.moe_layer(*args, y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    Hh.check_route(plan.layer_tensor(0), plan.layer_tensor(1), ref["topk_idx"], ref["topk_w"])
    ws = w.with_(E=w.E * S, K=w.K * S)
    Hh.check_dispatch(ws, plan.P, x, ref["topk_idx"], ref, plan.layer_tensor(2), plan.layer_tensor(3),
                      plan.layer_tensor(4), plan.layer_tensor(5), plan.layer_tensor(6))
    Hh.assert_output_close(Hh.to_host_f64(y), ref["y"], w.dtype)
    plain = Hh.make_plan(w, mode)
    y2 = torch.empty_like(y)
    plain.moe_layer(*args, y2)
    torch.cuda.synchronize()
    Hh.assert_output_close(Hh.to_host_f64(y), Hh.to_host_f64(y2), w.dtype, "with and without TP shards")


def test_tp_shards_with_overlap_and_push_combine():
    w, S = TP_CASES[1]
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd, tp_shards=S)
    args = [Hh.to_dev(a) for a in (x, wr, bias, wg, wu, wd)]
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_ORDERED, tp_shards=S, overlap=1, combine_mode=1)
    y = torch.empty((w.T, w.H), dtype=torch.bfloat16, device="cuda")
    plan.moe_layer(*args, y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    Hh.assert_output_close(Hh.to_host_f64(y), ref["y"], w.dtype)


def test_tp_shards_limits_are_refused_on_the_host():
    for cfg, code in [(B.make_config(64, 128, 8, 2, 2, 100, BF16, tp_shards=3), -1),     # F % S != 0
                      (B.make_config(64, 128, 128, 2, 2, 64, BF16, tp_shards=4), -3),    # E*S > 256
                      (B.make_config(64, 128, 64, 2, 16, 64, BF16, tp_shards=4), -3)]:   # K*S > 32
        with pytest.raises(B.MoeError) as ei:
            B.moe_workspace_bytes(cfg)
        assert ei.value.code == code


# ------------------------------------------------------------------ random small shapes
def _random_workloads(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        dtype = BF16 if rng.random() < 0.7 else FP32
        q = 8 if dtype == BF16 else 4                       # row pitch must be a multiple of 16 bytes
        E = int(rng.choice([1, 2, 3, 5, 8, 12, 24, 40, 64, 100, 256]))
        R = int(rng.choice([r for r in (1, 2, 3, 4, 5, 8) if E % r == 0]))
        K = int(rng.integers(1, min(E, 8) + 1))
        out.append(inputs.Workload(f"rand{i}", T=int(rng.integers(1, 400)), H=q * int(rng.integers(2, 40)), E=E, R=R,
                                   K=K, F=q * int(rng.integers(2, 40)), dtype=dtype,
                                   zipf_s=float(rng.choice([0.0, 1.0])), seed=int(rng.integers(0, 1000))))
    return out


@pytest.mark.parametrize("w", _random_workloads(24, 2024), ids=lambda w: f"{w.name}_T{w.T}_H{w.H}_E{w.E}_K{w.K}_F{w.F}_d{w.dtype}")
def test_random_small_layers_match_oracle(w):
    """Seeded random small shapes (ragged T, K = 1 ... 8, E from 1 to 256, odd H and F multiples, both
    dtypes, biased and unbiased routers), every dispatch scheme, whole layer against the oracle."""
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)
    for mode in MODES:
        plan = Hh.make_plan(w, mode)
        y = torch.empty((w.T, w.H), dtype=Hh.el_dtype(w), device="cuda")
        plan.moe_layer(Hh.to_dev(x), Hh.to_dev(wr), Hh.to_dev(bias), Hh.to_dev(wg), Hh.to_dev(wu), Hh.to_dev(wd), y)
        torch.cuda.synchronize()
        assert plan.moe_last_status() == (0, 0)
        Hh.check_route(plan.layer_tensor(0), plan.layer_tensor(1), ref["topk_idx"], ref["topk_w"])
        Hh.check_dispatch(w, plan.P, x, ref["topk_idx"], ref, plan.layer_tensor(2), plan.layer_tensor(3),
                          plan.layer_tensor(4), plan.layer_tensor(5), plan.layer_tensor(6))
        Hh.assert_output_close(Hh.to_host_f64(y), ref["y"], w.dtype)


@pytest.mark.parametrize("w", [w for w in _random_workloads(24, 2024) if w.dtype == BF16][:10],
                         ids=lambda w: f"{w.name}_T{w.T}_H{w.H}_E{w.E}_K{w.K}_F{w.F}")
def test_random_small_layers_variants_agree_bit_for_bit(w):
    """The variants of the bf16 layer do the same arithmetic in the same order per output element - ordered
    dispatch with the dispatch inside the expert launch, push-style combine, both together - so on the same
    seeded random shapes their y must equal the plain ordered layer's y bit for bit (which the test above holds
    against the oracle)."""
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    args = [Hh.to_dev(a) for a in (x, wr, bias, wg, wu, wd)]
    ys = []
    for kw in ({}, {"overlap": 1}, {"combine_mode": 1}, {"overlap": 1, "combine_mode": 1}):
        plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_ORDERED, **kw)
        y = torch.full((w.T, w.H), 7.0, dtype=torch.bfloat16, device="cuda")
        for _ in range(2):
            plan.moe_layer(*args, y)
        torch.cuda.synchronize()
        assert plan.moe_last_status() == (0, 0), kw
        ys.append(y)
    for kw, y in zip(("overlap", "push", "overlap + push"), ys[1:]):
        assert torch.equal(y, ys[0]), kw


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dtype", [BF16, FP32])
def test_empty_batch_is_a_legal_call(mode, dtype):
    """T = 0: every entry point accepts it, launches nothing that could touch a row, reports no error."""
    w = inputs.Workload("empty", T=0, H=128, E=8, R=2, K=2, F=128, dtype=dtype)
    _, wr, bias, wg, wu, wd = Hh.oracle_inputs(w.with_(T=4))
    plan = Hh.make_plan(w, mode)
    el = Hh.el_dtype(w)
    x = torch.empty((0, w.H), dtype=el, device="cuda")
    y = torch.empty((0, w.H), dtype=el, device="cuda")
    idx = torch.empty((0, w.K), dtype=torch.int32, device="cuda")
    tw = torch.empty((0, w.K), dtype=torch.float32, device="cuda")
    dwr, dwg, dwu, dwd = (Hh.to_dev(a) for a in (wr, wg, wu, wd))
    plan.moe_route(x, dwr, None, idx, tw)
    rows = plan.P * 128
    recv = torch.full((rows, w.H), 3.0, dtype=el, device="cuda")
    cnt = torch.full((w.E,), 9, dtype=torch.int32, device="cuda")
    te = torch.full((plan.P,), 9, dtype=torch.int32, device="cuda")
    src = torch.full((rows,), 9, dtype=torch.int32, device="cuda")
    slot = torch.empty((0, w.K), dtype=torch.int32, device="cuda")
    plan.moe_dispatch(x, idx, recv, cnt, te, src, slot)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    assert cnt.eq(0).all() and te.eq(-1).all() and recv.eq(3.0).all()      # nobody owns a tile, no row was written
    out_rows = torch.full((rows, w.H), 5.0, dtype=el, device="cuda")
    plan.moe_expert_ffn(recv, te, dwg, dwu, dwd, out_rows)
    plan.moe_combine(out_rows, slot, tw, y)
    plan.moe_layer(x, dwr, None, dwg, dwu, dwd, y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    assert out_rows.eq(5.0).all()                                          # no tile, no expert work


@pytest.mark.parametrize("dtype", [BF16, FP32])
def test_combine_treats_a_slot_beyond_the_pool_as_absent(dtype):
    """slot_of entries at or beyond the pool's rows (what an abandoned dispatch can leave behind) add nothing
    and are never used as an address: y is the weighted sum over the valid slots only."""
    w = inputs.Workload("bad_slots", T=64, H=256, E=8, R=2, K=4, F=128, dtype=dtype)
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_PAGED)
    rows = plan.P * 128
    g = torch.Generator(device="cuda").manual_seed(5)
    pool = torch.randn((rows, w.H), device="cuda", generator=g).to(Hh.el_dtype(w))
    slot = torch.randint(0, rows, (w.T, w.K), device="cuda", generator=g, dtype=torch.int32)
    slot[::3, 1] = rows               # first row past the pool
    slot[1::3, 2] = 2 ** 31 - 1       # as far out as an int goes
    slot[2::3, 0] = -1                # a dropped assignment
    tw = torch.rand((w.T, w.K), device="cuda", generator=g)
    y = torch.empty((w.T, w.H), dtype=Hh.el_dtype(w), device="cuda")
    plan.moe_combine(pool, slot, tw, y)
    torch.cuda.synchronize()
    valid = (slot >= 0) & (slot < rows)
    want = (pool.double()[slot.clamp(0, rows - 1).long()] * (tw.double() * valid).unsqueeze(-1)).sum(1)
    tol = 2.0 ** -7 if dtype == BF16 else 1e-5
    assert torch.allclose(y.double(), want, rtol=tol, atol=tol)


def test_pipelined_host_steps_match_single_steps():
    """moe_layer_host_submit / _wait with two steps in flight: five batches, each result identical to
    the same batch run alone through moe_layer (bit for bit: same kernels, same order)."""
    w = SMALL[3]
    _, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    dwr, dbias, dwg, dwu, dwd = (Hh.to_dev(a) for a in (wr, bias, wg, wu, wd))
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_PAGED)
    xs = [inputs.make_x(w.with_(seed=10 + i)) for i in range(5)]
    hx = [torch.from_numpy(x.view(np.int16)).pin_memory() for x in xs]
    hy = [torch.empty_like(h).pin_memory() for h in hx]
    tickets = []
    for i in range(5):
        tickets.append(plan.moe_layer_host_submit(hx[i], dwr, dbias, dwg, dwu, dwd, hy[i]))
        if i >= 1:
            plan.moe_layer_host_wait(tickets[i - 1])
    plan.moe_layer_host_wait(tickets[-1])
    assert tickets == list(range(5)) and plan.moe_last_status() == (0, 0)
    for i in range(5):
        y = torch.empty((w.T, w.H), dtype=torch.bfloat16, device="cuda")
        plan.moe_layer(Hh.to_dev(xs[i]), dwr, dbias, dwg, dwu, dwd, y)
        torch.cuda.synchronize()
        assert np.array_equal(hy[i].numpy().view(np.uint16), Hh.to_host_bits(y)), f"step {i}"


def test_layer_output_is_bit_identical_across_runs_and_dispatch_schemes():
    """Arrival order changes where a row sits, not what is computed for it: a row's GEMM result does not
    depend on its position in a tile and combine sums in ascending k, so y is the same bytes in every
    dispatch scheme and in every run, although the atomic schemes place rows in a different order each time."""
    w = SMALL[5]   # 256 experts, top-8, skewed
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    dev = [Hh.to_dev(a) for a in (x, wr, bias, wg, wu, wd)]
    outs, orders = [], []
    for mode in MODES:
        plan = Hh.make_plan(w, mode)
        for _ in range(3):
            y = torch.empty((w.T, w.H), dtype=torch.bfloat16, device="cuda")
            plan.moe_layer(*dev, y)
            torch.cuda.synchronize()
            outs.append(Hh.to_host_bits(y).tobytes())
            orders.append(plan.layer_tensor(6).cpu().numpy().tobytes())
    assert len(set(outs)) == 1
    assert len(set(orders)) > 1     # the placements did differ (scan vs atomic at the least)


def test_overlapped_launch_many_runs_same_bytes():
    """Forty runs of the overlapped launch on a layer with hot and cold experts (several tiles per hot expert, the
    narrow form for the cold ones, two expert launches): every run must give the bytes of the stream-ordered layer,
    with the receive pool refilled with 1e30 before each run - a consumer that started a tile too early, or a
    counter left over from the run before, would change them."""
    w = inputs.Workload("overlap_soak", T=3000, H=1024, E=48, R=4, K=4, F=512, dtype=BF16, zipf_s=1.0, seed=9)
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    dev = [Hh.to_dev(a) for a in (x, wr, bias, wg, wu, wd)]
    base = Hh.make_plan(w, B.DISPATCH_ATOMIC_ORDERED, ffn_split=1)
    y0 = torch.empty((w.T, w.H), dtype=torch.bfloat16, device="cuda")
    base.moe_layer(*dev, y0)
    torch.cuda.synchronize()
    assert base.moe_last_status() == (0, 0)
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_ORDERED, overlap=1, ffn_split=1)
    y = torch.empty_like(y0)
    for i in range(40):
        plan.layer_tensor(2).fill_(1.0e30)
        y.fill_(3.0)
        plan.moe_layer(*dev, y)
        torch.cuda.synchronize()
        assert plan.moe_last_status() == (0, 0), i
        assert torch.equal(y, y0), i


def _route_only(w, x, wr, bias, **kw):
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_PAGED, **kw)
    idx = torch.empty((w.T, w.K), dtype=torch.int32, device="cuda")
    tw = torch.empty((w.T, w.K), dtype=torch.float32, device="cuda")
    plan.moe_route(Hh.to_dev(x), Hh.to_dev(wr), Hh.to_dev(bias), idx, tw)
    torch.cuda.synchronize()
    return plan, idx, tw


@pytest.mark.parametrize("case", ["zero_rows", "equal_experts", "near_ties"])
def test_router_filter_degenerate_rows(case):
    """The tensor-core filter of the wide router where its candidate sets are as large as they get: tokens that are
    all zero (every logit equal: all 256 experts are candidates, the picks are experts 0..K-1), experts with identical
    weight rows (exact ties decided by index), and logits a few ulps apart."""
    w = inputs.Workload("filter_" + case, T=150, H=512, E=256, R=8, K=8, F=8, dtype=BF16, identity_experts=True, seed=4)
    x, wr, bias, *_ = Hh.oracle_inputs(w, with_experts=False)
    x, wr = x.copy(), wr.copy()
    if case == "zero_rows":
        x[::3] = 0
    elif case == "equal_experts":
        wr[1::2] = wr[0::2]                 # experts 2i and 2i+1 are the same row: every logit comes twice
    else:
        wr[:] = wr[0]                        # all experts alike ...
        wr[:, 0] = inputs.fp32_to_bf16_bits(np.linspace(-1e-2, 1e-2, w.E).astype(np.float32))   # ... but for one column
    _, idx, tw = _route_only(w, x, wr, None)
    ridx, rw, _ = oracle.route(x, wr, None, w.K, w.dtype)
    Hh.check_route(idx, tw, ridx, rw)
    # and the plain chains-for-everybody router gives the same
    _, idx2, tw2 = _route_only(w, x, wr, None, route_filter=-1)
    assert torch.equal(idx, idx2)


def test_router_filter_with_a_tiny_wait_limit_reports_or_routes():
    """Every wait of the two filter kernels is bounded.  With a limit of a nanosecond a wait either still finds its
    copy landed (a poll takes longer than that) or runs out: then the kernels give up by themselves and the status says
    so.  Never a hang, never a wrong pick without a status; a plan with the normal limit routes correctly afterwards."""
    w = inputs.Workload("filter_timeout", T=2048, H=2048, E=256, R=8, K=8, F=8, dtype=BF16, identity_experts=True)
    x, wr, bias, *_ = Hh.oracle_inputs(w, with_experts=False)
    ridx, rw, _ = oracle.route(x, wr, bias, w.K, w.dtype)
    plan, idx, tw = _route_only(w, x, wr, bias, wait_limit_ns=1)
    code, detail = plan.moe_last_status()
    if code == 0:
        Hh.check_route(idx, tw, ridx, rw)
    else:
        assert code == -6 and detail in (3, 4, 5), (code, detail)
    plan2, idx2, tw2 = _route_only(w, x, wr, bias)
    assert plan2.moe_last_status() == (0, 0)
    Hh.check_route(idx2, tw2, ridx, rw)
