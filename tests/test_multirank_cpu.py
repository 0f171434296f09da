"""The N > 1 plumbing of bench.py on CPU: two gloo ranks.  The hot path does not shard (replicas
only), so what there is to check is the max-over-ranks timing, the whole-job aggregate, and that
the reference arm runs on rank 0 alone under a multi-rank launch."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = [10.0 + 5.0 * rank, 3.0 - rank]         # rank 1 is slower on the first, faster on the second
    red = bench.max_over_ranks(ms)
    dist.barrier()
    out.put((rank, red, bench.whole_job_tokens_per_s(4096, world, red[0])))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    for rank, red, value in got:
        assert red == [15.0, 3.0]                                  # max over ranks, element-wise
        assert abs(value - 2 * 4096 / 15e-3) < 1e-6                # all ranks' tokens / slowest rank's time


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert bench.whole_job_tokens_per_s(100, 1, 10.0) == 10000.0


def test_reference_arm_prints_one_line_from_rank0_under_torchrun():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()),
           os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1", "--gpus", "2",
           "--steps", "2", "--warmup", "1"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["value"] > 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["e2e"]["h2d_bytes_per_step"] == 0
    assert rec["unit"] == "tokens/s" and rec["higher_is_better"] is True
