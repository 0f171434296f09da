"""Pins for the CPU oracle: every stage is checked against something that is not the oracle —
brute force, closed forms, invariants the paper states, or a library routine (torch CPU, fp64).

Paper hooks: the five steps of Section II-A; dense per-expert packing by a self-incrementing row
pointer and the address formula of Section IV-B; the source information that travels with each
row (Section IV-B, combine); the global completion count of Section IV-D (all T*K rows arrive).
"""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2605_05888_b200 import inputs

FP32, BF16 = inputs.FP32, inputs.BF16
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_storage(rng, shape, dtype, std=1.0):
    a = (rng.standard_normal(shape) * std).astype(np.float32)
    return inputs.fp32_to_bf16_bits(a) if dtype == BF16 else a


def widen(a, dtype):
    return inputs.bf16_bits_to_fp32(a).astype(np.float64) if dtype == BF16 else a.astype(np.float64)


# ---------------------------------------------------------------- step 1a: logits
@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_logits_identity_router_returns_x_exactly(dtype):
    # Closed form: H == E and Wr = I makes every chain x*1 + 0*..., so l == x bit for bit.
    rng = np.random.default_rng(1)
    E = H = 7
    x = rand_storage(rng, (5, H), dtype)
    eye = np.eye(E, dtype=np.float32)
    wr = inputs.fp32_to_bf16_bits(eye) if dtype == BF16 else eye
    lg = oracle.logits(x, wr, None, dtype)
    assert np.array_equal(lg, widen(x, dtype).astype(np.float32))


@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_logits_match_library_matmul(dtype):
    # Library routine: fp64 matmul in torch; a transposed operand or a dropped bias fails this.
    rng = np.random.default_rng(2)
    T, H, E = 9, 300, 6
    x, wr = rand_storage(rng, (T, H), dtype), rand_storage(rng, (E, H), dtype, 0.02)
    bias = rng.standard_normal(E).astype(np.float32)
    ref = (torch.from_numpy(widen(x, dtype)) @ torch.from_numpy(widen(wr, dtype)).T).numpy() + bias
    lg = oracle.logits(x, wr, bias, dtype)
    assert np.abs(lg - ref).max() < 1e-5
    lg0 = oracle.logits(x, wr, None, dtype)
    assert np.abs(lg0 - (ref - bias)).max() < 1e-5


def test_logits_chain_order_is_ascending_h():
    # (2^24 + 1) - 2^24 : the ascending chain loses the 1 (2^24+1 rounds to 2^24), giving 0;
    # the descending chain would give 1. Pins the summation order the bit-exact routing rests on.
    x = np.array([[16777216.0, 1.0, -16777216.0]], np.float32)
    wr = np.ones((1, 3), np.float32)
    assert oracle.logits(x, wr, None, FP32)[0, 0] == 0.0
    x = np.array([[-16777216.0, 16777216.0, 1.0]], np.float32)
    assert oracle.logits(x, wr, None, FP32)[0, 0] == 1.0


def test_logits_fused_multiply_add():
    # fl(a*b) != a*b here: a fused chain keeps the low bits of the product, mul-then-add loses them.
    a = np.float32(1 + 2 ** -12)
    x = np.array([[-1.0, a]], np.float32)
    wr = np.array([[np.float32(a * a), a]], np.float32)  # acc = -fl(a*a), then fma(a, a, acc) keeps a*a exact
    got = oracle.logits(x, wr, None, FP32)[0, 0]
    exact = float(a) * float(a) - float(np.float32(a * a))
    assert exact != 0.0 and got == np.float32(exact)


# ---------------------------------------------------------------- step 1b: top-k and weights
def brute_topk(l, K):
    order = sorted(range(len(l)), key=lambda e: (-float(l[e]), e))  # full sort, ties -> low index
    return order[:K]


def test_topk_exhaustive_tie_patterns():
    for E in range(1, 6):
        grid = np.array(list(itertools.product([-1.0, 0.0, 1.0], repeat=E)), np.float32)
        for K in range(1, E + 1):
            idx, w = oracle.topk(grid, K)
            for row, l in enumerate(grid):
                assert list(idx[row]) == brute_topk(l, K), (E, K, l)


def test_topk_negative_zero_ties_by_index():
    l = np.array([[0.0, -0.0, -0.0, 0.0]], np.float32)
    idx, _ = oracle.topk(l, 3)
    assert list(idx[0]) == [0, 1, 2]


def test_topk_random_vs_sort_and_invariants():
    rng = np.random.default_rng(3)
    T, E, K = 200, 60, 4
    l = rng.standard_normal((T, E)).astype(np.float32)
    l[:, 5] = l[:, 17]  # force ties
    idx, w = oracle.topk(l, K)
    for t in range(T):
        assert list(idx[t]) == brute_topk(l[t], K)
        assert len(set(idx[t])) == K
        sel = l[t, idx[t]]
        assert np.all(sel[:-1] >= sel[1:])
        rest = np.delete(l[t], idx[t])
        assert rest.max() <= sel[-1]


def test_weights_are_softmax_probabilities():
    rng = np.random.default_rng(4)
    T, E, K = 50, 16, 3
    l = (rng.standard_normal((T, E)) * 3).astype(np.float32)
    idx, w = oracle.topk(l, K)
    p = torch.softmax(torch.from_numpy(l.astype(np.float64)), dim=1).numpy()  # library routine
    ref = np.take_along_axis(p, idx.astype(np.int64), axis=1)
    assert np.abs(w - ref).max() < 1e-7
    idx2, w2 = oracle.topk(l, K, renormalize=1)
    assert np.array_equal(idx, idx2)
    assert np.abs(w2 - ref / ref.sum(1, keepdims=True)).max() < 1e-7
    assert np.abs(w2.sum(1) - 1).max() < 1e-6


def test_weights_closed_forms():
    E = 8
    idx, w = oracle.topk(np.full((3, E), 0.7, np.float32), E)  # K = E: whole softmax
    assert np.allclose(w, 1.0 / E, atol=1e-8) and np.allclose(w.sum(1), 1.0, atol=1e-6)
    assert [list(r) for r in idx] == [list(range(E))] * 3
    # two-expert logistic closed form: p0 = 1/(1+exp(-(l0-l1)))
    l = np.array([[2.0, -1.0]], np.float32)
    _, w = oracle.topk(l, 2)
    assert abs(w[0, 0] - 1 / (1 + np.exp(-3.0))) < 1e-7 and abs(w[0, 1] - 1 / (1 + np.exp(3.0))) < 1e-7


# ---------------------------------------------------------------- step 2: dispatch layout
@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_dispatch_invariants_and_stable_sort(dtype):
    rng = np.random.default_rng(5)
    T, H, E, R, K = 37, 16, 6, 3, 3
    x = rand_storage(rng, (T, H), dtype)
    idx = np.stack([rng.permutation(E)[:K] for _ in range(T)]).astype(np.int32)
    d = oracle.dispatch(x, idx, E, R, dtype)
    # every (token,k) assignment appears exactly once: slot_of is a bijection onto 0..T*K-1
    assert sorted(d["slot_of"].ravel()) == list(range(T * K))
    assert d["count"].sum() == T * K                                  # global completion count
    assert np.array_equal(d["count"], np.bincount(idx.ravel(), minlength=E))
    assert d["offset"][0] == 0 and np.array_equal(np.diff(d["offset"]), d["count"])
    assert np.array_equal(d["rank_count"], d["count"].reshape(R, E // R).sum(1))
    # source info travels with the row
    assert np.array_equal(d["src"][d["slot_of"].ravel()], np.arange(T * K))
    for t in range(T):
        for k in range(K):
            pos = d["slot_of"][t, k]
            assert d["offset"][idx[t, k]] <= pos < d["offset"][idx[t, k] + 1]  # in its expert's region
            assert d["recv"][pos].tobytes() == x[t].tobytes()                 # bytewise copy
    # textbook special case: a stable counting sort of the (t,k) pairs by expert
    assert np.array_equal(d["src"], np.argsort(idx.ravel(), kind="stable"))
    # each token appears exactly K times in the receive buffers
    assert np.array_equal(np.bincount(d["src"] // K, minlength=T), np.full(T, K))


def test_dispatch_empty_expert_and_single_expert():
    x = np.arange(12, dtype=np.float32).reshape(4, 3)
    idx = np.array([[2], [2], [2], [2]], np.int32)
    d = oracle.dispatch(x, idx, 4, 2, FP32)
    assert list(d["count"]) == [0, 0, 4, 0] and list(d["offset"]) == [0, 0, 0, 4, 4]
    assert list(d["rank_count"]) == [0, 4] and np.array_equal(d["recv"], x)


# ---------------------------------------------------------------- step 3: experts
def torch_swiglu(a, wg, wu, wd):
    a, wg, wu, wd = (torch.from_numpy(v) for v in (a, wg, wu, wd))
    return ((torch.nn.functional.silu(a @ wg.T) * (a @ wu.T)) @ wd.T).numpy()


@pytest.mark.parametrize("dtype", [FP32, BF16])
def test_ffn_single_expert_is_dense_swiglu_mlp(dtype):
    # E=1: the expert stage is an ordinary SwiGLU MLP; library routine in fp64 (F.silu, matmul).
    rng = np.random.default_rng(6)
    rows, H, F = 11, 24, 40
    a = rand_storage(rng, (rows, H), dtype)
    wg, wu, wd = (rand_storage(rng, s, dtype, 0.3) for s in ((F, H), (F, H), (H, F)))
    out = oracle.expert_ffn(a, np.array([0, rows], np.int32), [wg], [wu], [wd], dtype)
    ref = torch_swiglu(widen(a, dtype), widen(wg, dtype), widen(wu, dtype), widen(wd, dtype))
    assert np.abs(out - ref).max() < 1e-12 * max(1.0, np.abs(ref).max())


def test_ffn_uses_the_right_expert_and_skips_empty_ones():
    rng = np.random.default_rng(7)
    H, F, E = 8, 12, 4
    offset = np.array([0, 3, 3, 8, 10], np.int32)  # expert 1 empty: its weights are None
    a = rand_storage(rng, (10, H), FP32)
    ws = [tuple(rand_storage(rng, s, FP32, 0.5) for s in ((F, H), (F, H), (H, F))) for _ in range(E)]
    wg, wu, wd = ([w[i] if e != 1 else None for e, w in enumerate(ws)] for i in range(3))
    out = oracle.expert_ffn(a, offset, wg, wu, wd, FP32)
    for e in (0, 2, 3):
        r0, r1 = offset[e], offset[e + 1]
        ref = torch_swiglu(a[r0:r1].astype(np.float64), *(w.astype(np.float64) for w in ws[e]))
        assert np.abs(out[r0:r1] - ref).max() < 1e-12


def test_ffn_hand_probes():
    # one-hot input, small integer weights: every number below is worked by hand.
    H, F = 2, 2
    a = np.array([[1.0, 0.0]], np.float32)
    wg = np.array([[0.0, 5.0], [2.0, 7.0]], np.float32)   # g = (0, 2)
    wu = np.array([[3.0, 1.0], [4.0, 1.0]], np.float32)   # u = (3, 4)
    wd = np.array([[1.0, 1.0], [0.0, -1.0]], np.float32)
    out = oracle.expert_ffn(a, np.array([0, 1], np.int32), [wg], [wu], [wd], FP32)
    s1 = 2.0 / (1.0 + np.exp(-2.0)) * 4.0                 # silu(0)*3 = 0, silu(2)*4
    assert np.allclose(out[0], [s1, -s1], rtol=1e-14)
    zero = np.zeros_like(wg)
    assert np.all(oracle.expert_ffn(a, np.array([0, 1], np.int32), [zero], [wu], [wd], FP32) == 0)  # Wg=0 => s=0


# ---------------------------------------------------------------- steps 4+5: combine
def test_combine_identity_experts_returns_x_times_weight_sum():
    rng = np.random.default_rng(8)
    w = inputs.Workload("t", T=23, H=10, E=5, R=1, K=3, F=0, dtype=FP32, identity_experts=True)
    x = rand_storage(rng, (w.T, w.H), FP32)
    wr = rand_storage(rng, (w.E, w.H), FP32)
    r = oracle.layer(x, wr, None, None, None, None, w.E, w.R, w.K, FP32, identity_experts=True)
    ref = x.astype(np.float64) * r["topk_w"].astype(np.float64).sum(1, keepdims=True)
    assert np.abs(r["y"] - ref).max() < 1e-12
    full = oracle.layer(x, wr, None, None, None, None, w.E, w.R, w.E, FP32, identity_experts=True)
    assert np.abs(full["y"] - x).max() < 1e-6      # K = E: weights sum to one, y = x


def test_combine_is_linear_in_down_projection():
    rng = np.random.default_rng(9)
    T, H, E, K, F = 6, 8, 3, 2, 5
    x, wr = rand_storage(rng, (T, H), FP32), rand_storage(rng, (E, H), FP32)
    ws = [tuple(rand_storage(rng, s, FP32, 0.5) for s in ((F, H), (F, H), (H, F))) for _ in range(E)]
    y1 = oracle.layer(x, wr, None, *[[w[i] for w in ws] for i in range(3)], E, 1, K, FP32)["y"]
    y2 = oracle.layer(x, wr, None, [w[0] for w in ws], [w[1] for w in ws], [2 * w[2] for w in ws], E, 1, K, FP32)["y"]
    assert np.allclose(y2, 2 * y1, rtol=1e-12, atol=1e-15)


# ---------------------------------------------------------------- whole layer against the definition
def definition_layer(x, wr, bias, ws, K, renorm):
    """The layer as its definition, without any dispatch buffer: per token, pick experts by a full
    sort, weight by softmax, add w * FFN_e(x)."""
    T, H = x.shape
    E = wr.shape[0]
    y = np.zeros((T, H))
    for t in range(T):
        l = np.array([np.float32(sum(float(x[t, h]) * float(wr[e, h]) for h in range(H))) for e in range(E)])
        if bias is not None:
            l = (l + bias).astype(np.float32)
        picks = brute_topk(l, K)
        p = np.exp(l.astype(np.float64) - l.max())
        p /= p.sum()
        wsel = p[picks] / (p[picks].sum() if renorm else 1.0)
        for wk, e in zip(wsel, picks):
            wg, wu, wd = (v.astype(np.float64) for v in ws[e])
            g, u = wg @ x[t], wu @ x[t]
            y[t] += np.float32(wk) * (wd @ (g / (1 + np.exp(-g)) * u))
    return y


@pytest.mark.parametrize("renorm", [0, 1])
def test_whole_layer_exhaustive_tiny(renorm):
    # H == E, Wr = I: the logits ARE x, so enumerating x over a 3-value grid enumerates every
    # tie pattern of the router; all T = 3^E tokens go through the whole layer at once.
    rng = np.random.default_rng(10)
    for E, K in [(3, 1), (3, 2), (4, 2)]:
        H = E
        x = np.array(list(itertools.product([-1.0, 0.0, 1.0], repeat=E)), np.float32)
        wr = np.eye(E, dtype=np.float32)
        F = 3
        ws = [tuple(rng.integers(-2, 3, s).astype(np.float32) for s in ((F, H), (F, H), (H, F))) for _ in range(E)]
        r = oracle.layer(x, wr, None, *[[w[i] for w in ws] for i in range(3)], E, 1, K, FP32, renormalize=renorm)
        ref = definition_layer(x.astype(np.float64), wr, None, ws, K, renorm)
        assert np.abs(r["y"] - ref).max() < 1e-9


def test_whole_layer_random_with_bias_bf16():
    rng = np.random.default_rng(11)
    T, H, E, R, K, F = 12, 16, 6, 2, 3, 10
    x, wr = rand_storage(rng, (T, H), BF16), rand_storage(rng, (E, H), BF16, 0.3)
    bias = rng.standard_normal(E).astype(np.float32)
    ws = [tuple(rand_storage(rng, s, BF16, 0.3) for s in ((F, H), (F, H), (H, F))) for _ in range(E)]
    r = oracle.layer(x, wr, bias, *[[w[i] for w in ws] for i in range(3)], E, R, K, BF16)
    ws64 = [tuple(widen(v, BF16) for v in w) for w in ws]
    ref = definition_layer(widen(x, BF16), widen(wr, BF16).astype(np.float32), bias, ws64, K, 0)
    # the definition sums its logits in fp64, so the softmax weights differ in the 7th digit
    assert np.abs(r["y"] - ref).max() < 1e-6


# ---------------------------------------------------------------- hand-worked fixture
def test_golden_hand_worked_case():
    """tests/golden/fig2_shape_hand_case.txt: 4 experts on 2 ranks, top-2 (the set-up of the paper's
    Fig. 2), numbers worked by hand from the step definitions; the file states the derivation."""
    vals = {}
    with open(os.path.join(GOLDEN, "fig2_shape_hand_case.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=")
                vals[k.strip()] = np.array(eval(v, {"__builtins__": {}}, {}), dtype=np.float64)
    x = vals["x"].astype(np.float32)
    E, R, K = 4, 2, 2
    wr = np.eye(4, dtype=np.float32)
    r = oracle.layer(x, wr, None, None, None, None, E, R, K, FP32, identity_experts=True)
    assert np.array_equal(r["topk_idx"], vals["topk_idx"].astype(np.int32))
    assert np.abs(r["topk_w"] - vals["topk_w"]).max() < 1e-6
    assert np.array_equal(r["count"], vals["count"].astype(np.int32))
    assert np.array_equal(r["rank_count"], vals["rank_count"].astype(np.int32))
    assert np.array_equal(r["slot_of"], vals["slot_of"].astype(np.int32))
    assert np.array_equal(r["src"], vals["src"].astype(np.int32))
    assert np.abs(r["y"] - vals["y"]).max() < 1e-6


# ---------------------------------------------------------------- inputs module sanity
def test_inputs_are_slice_consistent_and_bf16_rounding_is_rne():
    a = inputs.normal(0, inputs.TAG_WG, 0, 5_000_000, 0.02, BF16)
    b = inputs.normal(0, inputs.TAG_WG, 4_194_000, 1000, 0.02, BF16)
    assert np.array_equal(a[4_194_000:4_195_000], b)
    f = np.array([1.0, 1.00390625, 1.01171875, 1.00390625 + 2 ** -20], np.float32)  # exact, tie->even, tie->even, just above a tie
    assert list(inputs.fp32_to_bf16_bits(f)) == [0x3F80, 0x3F80, 0x3F82, 0x3F81]
    t = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().astype(np.uint16)
    assert np.array_equal(inputs.fp32_to_bf16_bits(f), t)
    big = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    t = torch.from_numpy(big).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(inputs.fp32_to_bf16_bits(big), t)


# ---------------------------------------------------------------- expert + tensor parallelism (Section VII)
@pytest.mark.parametrize("dtype", [FP32, BF16])
@pytest.mark.parametrize("S", [2, 4])
def test_tp_shards_change_the_bookkeeping_but_not_the_result(S, dtype):
    """SwiGLU acts per FFN column and the down projection is a sum over FFN columns, so cutting an expert into S
    slices of its width and adding the slices' outputs gives the expert's output: the layer with TP shards must
    equal the plain layer (fp64: to rounding).  A slice taken from the wrong matrix axis, a pick's weight not
    carried to its shards, or a row missing from a shard's region breaks the equality.  The bookkeeping is that
    of E*S experts: every shard of a picked expert receives the row."""
    w = inputs.Workload("tp", T=37, H=24, E=6, R=3, K=2, F=16 * S, dtype=dtype, zipf_s=1.0, seed=4)
    x = inputs.make_x(w)
    wr, bias = inputs.make_router(w)
    wg, wu, wd = (list(a) for a in inputs.make_all_expert_weights(w))
    plain = oracle.layer(x, wr, bias, wg, wu, wd, w.E, w.R, w.K, dtype)
    tp = oracle.layer(x, wr, bias, wg, wu, wd, w.E, w.R, w.K, dtype, tp_shards=S)
    assert np.abs(tp["y"] - plain["y"]).max() <= 1e-12 * np.abs(plain["y"]).max()
    assert tp["topk_idx"].shape == (w.T, w.K * S)
    assert np.array_equal(tp["topk_idx"] // S, np.repeat(plain["topk_idx"], S, axis=1))
    assert np.array_equal(tp["topk_idx"] % S, np.tile(np.arange(S), (w.T, w.K)))
    assert np.array_equal(tp["topk_w"], np.repeat(plain["topk_w"], S, axis=1))
    assert np.array_equal(tp["count"], np.repeat(plain["count"], S))            # every shard gets every row of its expert
    assert tp["count"].sum() == w.T * w.K * S
    rows = tp["recv"][tp["slot_of"].ravel()]
    assert rows.tobytes() == np.repeat(x, w.K * S, axis=0).tobytes()
