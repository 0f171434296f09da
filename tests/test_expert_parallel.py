"""Real expert parallelism (tokens split along the sequence, experts across the ranks; paper Section II-A and
III-B): the partition, the address-centric baseline exchange on two gloo ranks (CPU), and the destination-
agnostic peer dispatch kernel with the ranks run one after the other on one GPU (every "peer" pointer is local
memory there; the kernel waits for nobody, so the ranks need not run at the same time)."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2605_05888_b200 import ep, inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def global_problem(T, H, E, K, R, seed=3):
    w = inputs.Workload("ep", T=T, H=H, E=E, R=R, K=K, F=8, dtype=inputs.BF16, zipf_s=1.0, seed=seed)
    x = inputs.make_x(w)
    wr, bias = inputs.make_router(w)
    idx, _, _ = oracle.route(x, wr, bias, K, w.dtype)
    return w, x, idx


def test_partition_covers_tokens_and_experts_once():
    T, E, R = 96, 12, 4
    toks, exps = zip(*(ep.partition(T, E, R, r) for r in range(R)))
    assert sorted(t for rng in toks for t in rng) == list(range(T))
    assert sorted(e for rng in exps for e in rng) == list(range(E))
    assert all(ep.owner_of(torch.tensor(list(exps[r])), E, R).eq(r).all() for r in range(R))
    with pytest.raises(ValueError):
        ep.partition(10, 12, 4, 0)


def _baseline_worker(rank, world, port, T, H, E, K, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w, x, idx = global_problem(T, H, E, K, world)
    toks, _ = ep.partition(T, E, world, rank)
    xl = torch.from_numpy(x[toks.start:toks.stop].view(np.int16))
    il = torch.from_numpy(idx[toks.start:toks.stop])
    got = ep.baseline_dispatch(xl, il, E)
    out.put((rank, got["rows"].numpy(), got["src"].numpy(), got["count"].numpy()))
    dist.barrier()
    dist.destroy_process_group()


def test_baseline_exchange_two_gloo_ranks_equals_the_oracle_dispatch():
    """Counts -> all-to-all of counts -> all-to-all of rows between two CPU processes: each rank ends up with
    exactly the rows the oracle's dispatch puts into its experts' regions, in (token, k) order."""
    T, H, E, K, R = 64, 16, 8, 2, 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = free_port()
    procs = [ctx.Process(target=_baseline_worker, args=(r, R, port, T, H, E, K, q)) for r in range(R)]
    for p in procs:
        p.start()
    got = {r: rest for r, *rest in (q.get(timeout=180) for _ in procs)}
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    w, x, idx = global_problem(T, H, E, K, R)
    ref = oracle.dispatch(x, idx, E, R, w.dtype)
    epr = E // R
    for r in range(R):
        rows, src, count = got[r]
        lo, hi = ref["offset"][r * epr], ref["offset"][(r + 1) * epr]
        assert np.array_equal(count, ref["count"][r * epr:(r + 1) * epr])
        assert rows.view(np.uint16).tobytes() == ref["recv"][lo:hi].tobytes()
        # the source id names (source rank, local token, k); with equal shares that is the global t*K+k
        assert np.array_equal(src, ref["src"][lo:hi])
        assert count.sum() == ref["rank_count"][r]


@pytest.mark.gpu
@pytest.mark.parametrize("R", [2, 4])
def test_peer_dispatch_kernel_ranks_run_one_after_the_other_on_one_gpu(R):
    """moe_dispatch_ep through the C ABI: every rank's call takes slots from the owners' allocation pointers and
    stores its rows into the owners' regions.  After all ranks ran: per expert the rows (sorted by source id) are
    the oracle's, counts and status counters are exact, slot_of finds every row again."""
    from paper_2605_05888_b200 import binding as B
    T, H, E, K = 512, 256, 16, 4
    w, x, idx = global_problem(T, H, E, K, R)
    ref = oracle.dispatch(x, idx, E, R, w.dtype)
    Tl, epr, cap = T // R, E // R, 512
    bufs = [ep.make_receive_buffers(E, R, H, cap, torch.bfloat16, "cuda") for _ in range(R)]
    for b in bufs:
        b["recv"].fill_(7.0)
    cfg = B.make_config(Tl, H, E, R, K, 8, inputs.BF16)
    slot_of = []
    for r in range(R):
        toks, _ = ep.partition(T, E, R, r)
        xl = torch.from_numpy(x[toks.start:toks.stop]).view(torch.int16).cuda().view(torch.bfloat16)
        il = torch.from_numpy(idx[toks.start:toks.stop]).cuda()
        so = torch.empty((Tl, K), dtype=torch.int32, device="cuda")
        status = torch.full((2,), 9, dtype=torch.int32, device="cuda")
        B.moe_dispatch_ep(cfg, r, bufs, cap, xl, il, so, status)
        torch.cuda.synchronize()
        assert status.cpu().tolist() == [0, 0]
        slot_of.append(so.cpu().numpy())
    slot = np.concatenate(slot_of)                      # [T, K] global row numbers: owner * epr * cap + row
    for r in range(R):
        b = bufs[r]
        cnt = b["row_pointer"].cpu().numpy()
        assert np.array_equal(cnt, ref["count"][r * epr:(r + 1) * epr])
        assert int(b["rows_done"][0]) == ref["rank_count"][r]
        src = b["src_info"].cpu().numpy()
        recv = b["recv"].view(torch.int16).cpu().numpy().view(np.uint16)
        tiles = b["tile_count"].cpu().numpy().reshape(epr, cap // 128)
        for le in range(epr):
            e = r * epr + le
            n = cnt[le]
            s = src[le * cap: le * cap + n]                              # dense from the region's start
            assert (src[le * cap + n:(le + 1) * cap] == -1).all()
            order = np.argsort(s, kind="stable")
            lo = ref["offset"][e]
            assert np.array_equal(s[order], ref["src"][lo:lo + n])       # equal shares: (rank*Tl + t)*K + k == t_global*K + k
            assert recv[le * cap: le * cap + n][order].tobytes() == ref["recv"][lo:lo + n].tobytes()
            assert tiles[le].sum() == n and (tiles[le] == np.clip(n - 128 * np.arange(cap // 128), 0, 128)).all()
    # slot_of <-> src_info across ranks
    owner, row = slot // (epr * cap), slot % (epr * cap)
    assert np.array_equal(owner, idx // epr)
    for r in range(R):
        m = owner == r
        assert np.array_equal(bufs[r]["src_info"].cpu().numpy()[row[m]], np.arange(T * K).reshape(T, K)[m])


@pytest.mark.gpu
def test_peer_dispatch_reports_a_full_region():
    from paper_2605_05888_b200 import binding as B
    T, H, E, K, R = 300, 64, 4, 1, 2
    x = inputs.make_x(inputs.Workload("epo", T=T, H=H, E=E, R=R, K=K, F=8, dtype=inputs.BF16))
    idx = np.full((T, K), 3, np.int32)                                   # every row to expert 3 (rank 1)
    bufs = [ep.make_receive_buffers(E, R, H, 128, torch.bfloat16, "cuda") for _ in range(R)]
    guard = torch.full((2 * 128 + 64, H), 5.0, dtype=torch.bfloat16, device="cuda")
    bufs[1]["recv"] = guard[:2 * 128]
    so = torch.empty((T, K), dtype=torch.int32, device="cuda")
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    cfg = B.make_config(T, H, E, R, K, 8, inputs.BF16)
    xl = torch.from_numpy(x).view(torch.int16).cuda().view(torch.bfloat16)
    B.moe_dispatch_ep(cfg, 0, bufs, 128, xl, torch.from_numpy(idx).cuda(), so, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [-5, 3]
    s = so.cpu().numpy().ravel()
    assert (s >= 0).sum() == 128 and (s == -1).sum() == T - 128
    assert int(bufs[1]["rows_done"][0]) == T and torch.all(guard[2 * 128:] == 5.0)


def ep_layer_problem(T, H, E, K, F, R, dtype):
    import parity_helpers as Hh
    w = inputs.Workload("ep_layer", T=T, H=H, E=E, R=R, K=K, F=F, dtype=dtype, zipf_s=0.8, seed=11)
    return (w,) + Hh.oracle_inputs(w)


@pytest.mark.gpu
@pytest.mark.parametrize("R,dtype", [(2, inputs.BF16), (4, inputs.BF16), (2, inputs.FP32)])
def test_expert_parallel_layer_ranks_run_phase_by_phase_on_one_gpu(R, dtype):
    """The whole destination-agnostic layer over R ranks - route, peer dispatch, experts on the owner, result rows
    pushed back to the source rank's staging buffer, weighted sum - against the oracle's plain layer on the whole
    batch.  The ranks are objects in one process and run phase by phase; every peer pointer is local memory."""
    import parity_helpers as Hh
    T, H, E, K, F = 384, 256, 8, 2, 128
    w, x, wr, bias, wg, wu, wd = ep_layer_problem(T, H, E, K, F, R, dtype)
    Tl, epr = T // R, E // R
    ranks = [ep.EpRank(r, R, Tl, H, E, K, F, dtype) for r in range(R)]
    xs = [Hh.to_dev(np.ascontiguousarray(x[r * Tl:(r + 1) * Tl]), dtype) for r in range(R)]
    dwr, dbias = Hh.to_dev(wr, dtype), Hh.to_dev(bias)
    shard = lambda m: [Hh.to_dev(np.ascontiguousarray(m[r * epr:(r + 1) * epr]), dtype) for r in range(R)]
    ys = [torch.empty((Tl, H), dtype=ranks[0].el, device="cuda") for _ in range(R)]
    ref = Hh.oracle_layer_for(w, x, wr, bias, wg, wu, wd)
    for _ in range(2):                       # a second step finds every counter back in its start state
        for y in ys:
            y.zero_()
        ep.run_in_process(ranks, xs, dwr, dbias, shard(wg), shard(wu), shard(wd), ys)
        got = np.concatenate([Hh.to_host_f64(y) for y in ys])
        Hh.assert_output_close(got, ref["y"], dtype, f"EP layer, R = {R}")
    for r, rk in enumerate(ranks):
        assert int(rk.own["rows_back"][0]) == Tl * K
        assert np.array_equal(rk.expert_count.cpu().numpy(), ref["count"][r * epr:(r + 1) * epr])
        assert int(rk.own["rows_done"][0]) == ref["rank_count"][r]


@pytest.mark.gpu
@pytest.mark.parametrize("R", [2, 3])
def test_expert_parallel_layer_one_process_per_rank_through_cuda_ipc(R):
    """The same layer with one PROCESS per rank: the ranks exchange CUDA IPC handles of their receive and staging
    buffers over gloo and write into one another's memory with the peer kernels.  All processes share the one
    visible GPU, which is legal because no kernel waits for another rank's kernel; each rank checks its own tokens
    against the oracle and the exit codes carry the verdict."""
    import subprocess
    T, H, E, K, F = 96 * R, 256, 4 * R, 2, 128
    port = free_port()
    procs = []
    for r in range(R):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE=str(R), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.join(ROOT, "tests", "ep_worker.py"),
                                       *(str(v) for v in (T, H, E, K, F, inputs.BF16))], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = []
    for p in procs:
        try:
            out, _ = p.communicate(timeout=300)
        except subprocess.TimeoutExpired:
            p.kill()
            out, _ = p.communicate()
        outs.append(out)
    assert [p.returncode for p in procs] == [0] * R, "\n".join(o[-2000:] for o in outs)
