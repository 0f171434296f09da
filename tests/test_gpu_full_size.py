"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times (moe_layer,
paged atomic dispatch, tensor-core experts).

Routing and dispatch are compared with the oracle in full (bit-exact).  The expert FFN at these
sizes is 3-6 TFLOP, too much for the CPU oracle, so the combined output is compared on a sample of
tokens: tokens are independent, so the oracle layer run on x[sample] gives exactly the rows
y[sample] of the full batch.  The sample is drawn from the run's own slot_of so that EVERY used
128-row tile of the receive pool holds at least one compared row (every work item of the expert
kernel, whatever its form, contributes to a compared output), plus a seeded random sample.  Properties that hold at any size (identity experts give
x * sum_k w) cover the largest dispatch/combine sweep point.
"""
import numpy as np
import pytest
import torch

import oracle
import parity_helpers as Hh
from paper_2605_05888_b200 import binding as B
from paper_2605_05888_b200 import inputs

pytestmark = pytest.mark.gpu


def run_layer(w, mode, x, wr, bias, dwg, dwu, dwd):
    plan = Hh.make_plan(w, mode)
    y = torch.empty((w.T, w.H), dtype=Hh.el_dtype(w), device="cuda")
    plan.moe_layer(Hh.to_dev(x), Hh.to_dev(wr), Hh.to_dev(bias), dwg, dwu, dwd, y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    return plan, y


def check_full_routing_and_dispatch(w, plan, x, wr, bias):
    idx, tw, _ = oracle.route(x, wr, bias, w.K, w.dtype)
    Hh.check_route(plan.layer_tensor(0), plan.layer_tensor(1), idx, tw)
    d = oracle.dispatch(x, idx, w.E, w.R, w.dtype)
    Hh.check_dispatch(w, plan.P, x, idx, d, plan.layer_tensor(2), plan.layer_tensor(3), plan.layer_tensor(4),
                      plan.layer_tensor(5), plan.layer_tensor(6))
    return idx, d


def check_sampled_output(w, plan, y, x, wr, bias, wg, wu, wd, n_sample, seed=0):
    rng = np.random.default_rng(seed)
    slot = plan.layer_tensor(6).cpu().numpy()
    sample = Hh.tokens_covering_every_tile(slot, np.sort(rng.choice(w.T, size=n_sample, replace=False)))
    used = np.unique(slot // 128)
    assert np.array_equal(np.unique(slot[sample] // 128), used), "a used tile has no compared row"
    xs = np.ascontiguousarray(x[sample])
    ref = oracle.layer(xs, wr, bias, list(wg), list(wu), list(wd), w.E, w.R, w.K, w.dtype)
    got = Hh.to_host_f64(y[torch.from_numpy(sample).cuda()])
    Hh.assert_output_close(got, ref["y"], w.dtype, "sampled tokens")
    stored = oracle.layer(xs, wr, bias, list(wg), list(wu), list(wd), w.E, w.R, w.K, w.dtype, bf16_storage=True)
    Hh.assert_close_to_bf16_storage(got, stored, "sampled tokens")
    return sample.size, used.size


@pytest.mark.parametrize("mode", [B.DISPATCH_ATOMIC_PAGED, B.DISPATCH_SCAN, B.DISPATCH_ATOMIC_ORDERED])
def test_c2_mixtral_like_full_size(mode):
    w = inputs.C2
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    plan, y = run_layer(w, mode, x, wr, bias, Hh.to_dev(wg), Hh.to_dev(wu), Hh.to_dev(wd))
    _, d = check_full_routing_and_dispatch(w, plan, x, wr, bias)
    # near-uniform load (the recipe's forecast: every expert within a few percent of T*K/E)
    assert d["count"].min() > 0.9 * w.T * w.K / w.E and d["count"].max() < 1.1 * w.T * w.K / w.E
    check_sampled_output(w, plan, y, x, wr, bias, wg, wu, wd, 32)


@pytest.mark.parametrize("mode", [B.DISPATCH_ATOMIC_PAGED, B.DISPATCH_ATOMIC_ORDERED])
def test_c3_deepseek_like_full_size_skewed(mode):
    w = inputs.C3
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    plan, y = run_layer(w, mode, x, wr, bias, Hh.to_dev(wg), Hh.to_dev(wu), Hh.to_dev(wd))
    _, d = check_full_routing_and_dispatch(w, plan, x, wr, bias)
    # the Zipf bias really skews the load: hottest expert far above the mean, some experts below one tile
    assert d["count"].max() > 8 * w.T * w.K / w.E and (d["count"] < 128).sum() > 32
    check_sampled_output(w, plan, y, x, wr, bias, wg, wu, wd, 24)


@pytest.mark.parametrize("w", [inputs.C2, inputs.C3, inputs.C4], ids=lambda w: w.name)
def test_push_combine_full_size(w):
    """Push-style combine at the benchmark's sizes (every form of the expert kernel's final epilogue: full tiles,
    short last tiles, narrow single tiles): the same bytes in y as the gather path, and the oracle's output on a
    row of every used tile."""
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    args = [Hh.to_dev(a) for a in (x, wr, bias, wg, wu, wd)]
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_PAGED, combine_mode=1)
    y = torch.empty((w.T, w.H), dtype=Hh.el_dtype(w), device="cuda")
    plan.moe_layer(*args, y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    check_sampled_output(w, plan, y, x, wr, bias, wg, wu, wd, 16)
    gather = Hh.make_plan(w, B.DISPATCH_ATOMIC_PAGED)
    y2 = torch.empty_like(y)
    gather.moe_layer(*args, y2)
    torch.cuda.synchronize()
    assert torch.equal(y, y2)


@pytest.mark.parametrize("w", [inputs.C2, inputs.C3, inputs.C4], ids=lambda w: w.name)
def test_overlapped_launch_full_size(w):
    """Dispatch inside the expert kernel's launch (producer CTAs emit the tokens in ascending order, consumer
    CTAs start on a tile when its status counter reaches the rows it will hold) at the benchmark's sizes:
    routing and dispatch in full, output on a row of every used tile; and in one traced layer the first expert
    item begins before the last row is stored."""
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    plan = Hh.make_plan(w, B.DISPATCH_ATOMIC_ORDERED, overlap=1)
    y = torch.empty((w.T, w.H), dtype=Hh.el_dtype(w), device="cuda")
    args = [Hh.to_dev(a) for a in (x, wr, bias, wg, wu, wd)]
    plan.layer_tensor(2).fill_(1.0e30)     # a row consumed before it was stored would show in y
    plan.moe_layer(*args, y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    check_full_routing_and_dispatch(w, plan, x, wr, bias)
    check_sampled_output(w, plan, y, x, wr, bias, wg, wu, wd, 16)
    plan.moe_availability_trace(True)
    plan.layer_tensor(9).zero_()
    plan.moe_layer(*args, y)
    torch.cuda.synchronize()
    tr = plan.layer_tensor(8).cpu().numpy()
    items = plan.layer_tensor(9).cpu().numpy()
    started = items[items[:, 0] > 0]
    gemm1 = started[(started[:, 2] & 1) == 0]
    assert gemm1[:, 0].min() < tr[1], "no expert item began before the dispatch was over"


@pytest.mark.parametrize("mode", [B.DISPATCH_SCAN, B.DISPATCH_ATOMIC_STATIC, B.DISPATCH_ATOMIC_PAGED, B.DISPATCH_ATOMIC_ORDERED])
def test_c4_qwen_like_full_size(mode):
    w = inputs.C4
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    plan, y = run_layer(w, mode, x, wr, bias, Hh.to_dev(wg), Hh.to_dev(wu), Hh.to_dev(wd))
    check_full_routing_and_dispatch(w, plan, x, wr, bias)
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)      # small enough for the whole oracle layer
    Hh.assert_output_close(Hh.to_host_f64(y), ref["y"], w.dtype)
    stored = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd, bf16_storage=True)
    Hh.assert_close_to_bf16_storage(Hh.to_host_f64(y), stored)


@pytest.mark.parametrize("w", [inputs.PHI35, inputs.QWEN64], ids=lambda w: w.name)
def test_other_table2_shapes(w):
    """Phi-3.5-MoE and Qwen2-MoE (64 experts) shapes of the paper's Table II: routing and dispatch in full,
    output on sampled tokens."""
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    plan, y = run_layer(w, B.DISPATCH_ATOMIC_PAGED, x, wr, bias, Hh.to_dev(wg), Hh.to_dev(wu), Hh.to_dev(wd))
    check_full_routing_and_dispatch(w, plan, x, wr, bias)
    check_sampled_output(w, plan, y, x, wr, bias, wg, wu, wd, 32)


@pytest.mark.parametrize("mode", [B.DISPATCH_ATOMIC_PAGED, B.DISPATCH_ATOMIC_ORDERED])
@pytest.mark.parametrize("zipf", [0.0, 1.2])
def test_c5_sweep_point_8192_against_oracle(zipf, mode):
    w = inputs.C5(8192, zipf)
    x, wr, bias, *_ = Hh.oracle_inputs(w, with_experts=False)
    plan, y = run_layer(w, mode, x, wr, bias, None, None, None)
    idx, d = check_full_routing_and_dispatch(w, plan, x, wr, bias)
    _, tw, _ = oracle.route(x, wr, bias, w.K, w.dtype)
    ref = oracle.combine(oracle.identity_ffn(d["recv"], w.dtype), d["slot_of"], tw)
    Hh.assert_output_close(Hh.to_host_f64(y), ref, w.dtype)


@pytest.mark.parametrize("mode", [B.DISPATCH_SCAN, B.DISPATCH_ATOMIC_PAGED, B.DISPATCH_ATOMIC_ORDERED])
def test_c5_largest_sweep_point_properties(mode):
    """T = 65536 (8.5 GB moved per direction): checked by properties that hold at any size."""
    w = inputs.C5(65536, 1.2)
    x, wr, bias, *_ = Hh.oracle_inputs(w, with_experts=False)
    dx = Hh.to_dev(x)
    plan = Hh.make_plan(w, mode)
    y = torch.empty((w.T, w.H), dtype=torch.bfloat16, device="cuda")
    plan.moe_layer(dx, Hh.to_dev(wr), Hh.to_dev(bias), None, None, None, y)
    torch.cuda.synchronize()
    assert plan.moe_last_status() == (0, 0)
    idx, tw = plan.layer_tensor(0), plan.layer_tensor(1)
    cnt, te, src, slot = (plan.layer_tensor(i) for i in (3, 4, 5, 6))
    assert int(cnt.sum()) == w.T * w.K                                   # every row arrived
    assert torch.equal(cnt.long(), torch.bincount(idx.flatten().long(), minlength=w.E))
    flat = slot.flatten().long()
    assert torch.equal(src[flat].long(), torch.arange(w.T * w.K, device="cuda"))   # bijection with source info
    assert torch.equal(te[flat // 128], idx.flatten())                   # every row in a tile of its expert
    assert int((te >= 0).sum()) == int(((cnt + 127) // 128).sum())       # dense packing
    # sampled rows are byte copies of their token; sampled outputs equal x * sum_k w
    g = torch.Generator(device="cpu").manual_seed(0)
    a = torch.randint(0, w.T * w.K, (4096,), generator=g).cuda()
    recv = plan.layer_tensor(2)
    assert torch.equal(recv[flat[a]].view(torch.int16), dx[a // w.K].view(torch.int16))
    t = torch.randint(0, w.T, (2048,), generator=g).cuda()
    ref = (dx[t].double() * tw[t].double().sum(1, keepdim=True)).cpu().numpy()
    Hh.assert_output_close(Hh.to_host_f64(y[t]), ref, w.dtype)
    # sampled routing decisions against the oracle
    ts = np.sort(np.random.default_rng(1).choice(w.T, 256, replace=False))
    ridx, rw, _ = oracle.route(np.ascontiguousarray(x[ts]), wr, bias, w.K, w.dtype)
    Hh.check_route(idx[torch.from_numpy(ts).cuda()], tw[torch.from_numpy(ts).cuda()], ridx, rw)
