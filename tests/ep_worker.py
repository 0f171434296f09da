"""One rank of the multi-process expert-parallel layer test (started by tests/test_expert_parallel.py, one process
per rank, all on the visible GPU): builds the rank, maps the peers' buffers through CUDA IPC, runs one layer step
and compares this rank's tokens with the oracle.  Exit code 0 = parity."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

import oracle  # noqa: E402
import parity_helpers as Hh  # noqa: E402
from paper_2605_05888_b200 import ep, inputs  # noqa: E402


def main() -> int:
    rank, R = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    T, H, E, K, F, dtype = (int(v) for v in sys.argv[1:7])
    dist.init_process_group("gloo", rank=rank, world_size=R)
    w = inputs.Workload("ep_layer", T=T, H=H, E=E, R=R, K=K, F=F, dtype=dtype, zipf_s=0.8, seed=11)
    x, wr, bias, wg, wu, wd = Hh.oracle_inputs(w)
    toks, exps = ep.partition(T, E, R, rank)
    me = ep.EpRank(rank, R, T // R, H, E, K, F, dtype)
    group = ep.EpGroup(me)
    xl = Hh.to_dev(np.ascontiguousarray(x[toks.start:toks.stop]), dtype)
    dev = [Hh.to_dev(a, dtype) if a is not None else None for a in (wr, bias)]
    mine = [Hh.to_dev(np.ascontiguousarray(m[exps.start:exps.stop]), dtype) for m in (wg, wu, wd)]
    y = torch.empty((T // R, H), dtype=me.el, device="cuda")
    for _ in range(2):                                     # twice: the counters must return to their start state
        y.zero_()
        group.step(xl, dev[0], dev[1], *mine, y)
    ref = Hh.oracle_layer_for(w, x[toks.start:toks.stop], wr, bias, wg, wu, wd)
    ok = True
    try:
        Hh.assert_output_close(Hh.to_host_f64(y), ref["y"], dtype, f"rank {rank}")
        # every assignment of this rank's tokens came back: the counter other ranks raised says so
        assert int(me.own["rows_back"][0]) == (T // R) * K
        # and the rows this rank's experts received are the oracle's counts
        cnt = np.bincount(oracle.route(x, wr, bias, K, dtype)[0].ravel(), minlength=E)[exps.start:exps.stop]
        assert np.array_equal(me.expert_count.cpu().numpy(), cnt)
    except AssertionError as e:
        print(f"rank {rank}: {e}", flush=True)
        ok = False
    group.close()
    dist.destroy_process_group()
    return 0 if ok else 1


if __name__ == "__main__":
    sys.exit(main())
