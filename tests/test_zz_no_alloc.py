"""moe_dispatch_noalloc, the dispatch entry point for callers that cannot allocate device memory
(it keeps its scratch in a fixed array inside the library).

This file is collected last on purpose: a run that stops at the first failure has then already
run every other test.  It passes alone in a fresh process and after the other tests.

The entry point is called through the C ABI twice in a row with different routing, so the second
call meets the scratch array exactly as the first one left it.  Dispatch is byte and index work,
so every check is exact: each assignment's row is the bytes of its token (read through slot_of,
which removes the one freedom, the arrival order of rows inside an expert), it sits in a tile of
its expert, counts are a bincount of the routing, tiles are densely packed.  The ordinary
moe_dispatch is run on the same inputs and must agree on everything that is unique; and the warm
second call must leave the amount of free device memory exactly where it was.
"""
import numpy as np
import pytest
import torch

from paper_2605_05888_b200 import binding as B
from paper_2605_05888_b200 import inputs

pytestmark = pytest.mark.gpu


def dev_bf16(a):
    return torch.from_numpy(a).view(torch.int16).cuda().view(torch.bfloat16)


def buffers(P, w):
    rows = P * 128
    return dict(recv=torch.zeros((rows, w.H), dtype=torch.bfloat16, device="cuda"),
                cnt=torch.empty(w.E, dtype=torch.int32, device="cuda"),
                te=torch.empty(P, dtype=torch.int32, device="cuda"),
                src=torch.empty(rows, dtype=torch.int32, device="cuda"),
                slot=torch.empty((w.T, w.K), dtype=torch.int32, device="cuda"))


def canonical(b, w):
    """What is unique about a dispatch result: counts, and per assignment its row bytes and owner."""
    slot = b["slot"].cpu().numpy().ravel()
    assert slot.min() >= 0 and np.unique(slot).size == w.T * w.K
    src = b["src"].cpu().numpy()
    assert np.array_equal(src[slot], np.arange(w.T * w.K)) and (src >= 0).sum() == w.T * w.K
    rows = b["recv"].view(torch.int16).cpu().numpy()[slot]
    owner = b["te"].cpu().numpy()[slot // 128]
    tiles = np.bincount(b["te"].cpu().numpy()[b["te"].cpu().numpy() >= 0], minlength=w.E)
    return b["cnt"].cpu().numpy(), rows, owner, tiles


def test_noalloc_dispatch_moves_the_right_bytes_twice_in_a_row():
    w = inputs.Workload("noalloc", T=1500, H=512, E=32, R=4, K=4, F=64, dtype=inputs.BF16, zipf_s=1.0)
    x = inputs.make_x(w)
    dx = dev_bf16(x)
    cfg = B.make_config(w.T, w.H, w.E, w.R, w.K, w.F, w.dtype, dispatch_mode=B.DISPATCH_ATOMIC_PAGED)
    plan = B.Plan(cfg)
    status = torch.full((2,), 123, dtype=torch.int32, device="cuda")
    rng = np.random.default_rng(0)
    for call in range(2):
        # different routing each time: call 0 skewed to a few experts, call 1 spread over all of them
        hi = 6 if call == 0 else w.E
        idx = np.stack([rng.permutation(hi)[:w.K] for _ in range(w.T)]).astype(np.int32)
        didx = torch.from_numpy(idx).cuda()
        old, new = buffers(plan.P, w), buffers(plan.P, w)
        plan.moe_dispatch(dx, didx, old["recv"], old["cnt"], old["te"], old["src"], old["slot"])
        assert plan.moe_last_status() == (0, 0)
        torch.cuda.synchronize()
        free_before, torch_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        B.moe_dispatch_noalloc(cfg, dx, didx, new["recv"], new["cnt"], new["te"], new["src"], new["slot"], status)
        torch.cuda.synchronize()
        if call == 1:   # the warm call: the library took no device memory, through torch or past it
            assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == torch_before
        assert status.cpu().tolist() == [0, 0]
        c_new, r_new, o_new, t_new = canonical(new, w)
        # against the definition: row of assignment (t, k) == x[t] bytewise, in a tile of expert idx[t, k]
        assert r_new.tobytes() == np.repeat(x.view(np.int16), w.K, axis=0).tobytes()
        assert np.array_equal(o_new, idx.ravel())
        assert np.array_equal(c_new, np.bincount(idx.ravel(), minlength=w.E))
        assert np.array_equal(t_new, (c_new + 127) // 128)
        # and against the existing entry point
        c_old, r_old, o_old, t_old = canonical(old, w)
        assert np.array_equal(c_new, c_old) and r_new.tobytes() == r_old.tobytes()
        assert np.array_equal(o_new, o_old) and np.array_equal(t_new, t_old)


def test_noalloc_dispatch_rejects_sizes_beyond_its_scratch():
    cfg = B.make_config(16385, 128, 8, 1, 2, 64, inputs.BF16)
    dummy = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(B.MoeError) as ei:
        B.moe_dispatch_noalloc(cfg, dummy, dummy, dummy, dummy, dummy, dummy, dummy, dummy)
    assert ei.value.code == -8 and "scratch" in str(ei.value)
