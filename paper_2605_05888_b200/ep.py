"""Host side of real expert parallelism (R GPUs, one process per GPU): who owns what, the receive buffers a
rank offers to its peers, and the address-centric baseline the destination-agnostic dispatch is shown against.

Partition (Section II-A of the paper: tokens are split along the sequence, experts across the GPUs): rank r
holds tokens [r*T/R, (r+1)*T/R) and experts [r*E/R, (r+1)*E/R).

Two ways to get a row to its expert's GPU:
  * destination-agnostic (``binding.moe_dispatch_ep``): the producer takes a slot from the consumer's allocation
    pointer with a remote atomic and stores the row there; no rank tells any other rank counts or offsets.
  * the baseline (``baseline_dispatch`` below): the software mediation of Section III-A - every rank counts its
    rows per destination, the ranks exchange the counts, compute offsets, and only then move the rows with an
    all-to-all.  Written with torch.distributed collectives only, so it runs on NCCL between GPUs and on gloo
    between CPU processes (which is how it is tested).

Nothing here does arithmetic of the method; rows are moved as bytes.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def partition(T: int, E: int, R: int, rank: int) -> tuple[range, range]:
    """(token range, expert range) of `rank`.  T and E must be multiples of R."""
    if T % R or E % R or not 0 <= rank < R:
        raise ValueError("T and E must be multiples of R and 0 <= rank < R")
    return range(rank * T // R, (rank + 1) * T // R), range(rank * E // R, (rank + 1) * E // R)


def owner_of(expert: torch.Tensor, E: int, R: int) -> torch.Tensor:
    return expert // (E // R)


def make_receive_buffers(E: int, R: int, H: int, cap_rows: int, dtype: torch.dtype, device) -> dict:
    """The buffers one rank offers to its peers for ``moe_dispatch_ep``, in their start state."""
    epr = E // R
    return {"recv": torch.empty((epr * cap_rows, H), dtype=dtype, device=device),
            "row_pointer": torch.zeros(epr, dtype=torch.int32, device=device),
            "tile_count": torch.zeros(epr * cap_rows // 128, dtype=torch.int32, device=device),
            "src_info": torch.full((epr * cap_rows,), -1, dtype=torch.int32, device=device),
            "rows_done": torch.zeros(1, dtype=torch.int32, device=device)}


def baseline_dispatch(x_local: torch.Tensor, topk_idx_local: torch.Tensor, E: int, group=None) -> dict:
    """Address-centric dispatch: counts -> exchange of counts -> offsets -> all-to-all of rows.

    x_local [T_local, H], topk_idx_local [T_local, K] (int32, global expert ids), on this rank's device.
    Returns, for this rank's experts: rows [n, H] grouped by local expert (within an expert: by source rank, then
    (token, k)), src [n] = (source rank * T_local + t) * K + k, count [E/R] rows per local expert.
    """
    R = dist.get_world_size(group)
    rank = dist.get_rank(group)
    T, K = topk_idx_local.shape
    epr = E // R
    flat = topk_idx_local.reshape(-1).to(torch.int64)
    dest = flat // epr
    # stable order by (destination rank, expert): what the sender's scan + scatter produces
    order = torch.argsort(flat, stable=True)
    send_rows = x_local[order // K].contiguous()
    send_expert = (flat[order] % epr).to(torch.int32)
    send_src = ((rank * T) * K + order).to(torch.int32)
    send_counts = torch.bincount(dest, minlength=R).to(torch.int64)
    recv_counts = torch.empty_like(send_counts)
    dist.all_to_all_single(recv_counts, send_counts, group=group)             # the mediation step: exchange the counts
    n = int(recv_counts.sum())
    ins, outs = send_counts.tolist(), recv_counts.tolist()

    def exchange(t: torch.Tensor) -> torch.Tensor:
        # rows travel as bytes (every backend moves uint8; not every backend knows bf16 or int16)
        tb = t.contiguous().view(torch.uint8).reshape(t.shape[0], -1)
        out = torch.empty((n, tb.shape[1]), dtype=torch.uint8, device=t.device)
        dist.all_to_all_single(out, tb, output_split_sizes=outs, input_split_sizes=ins, group=group)
        return out.view(t.dtype).reshape((n,) + tuple(t.shape[1:]))

    rows, expert, src = exchange(send_rows), exchange(send_expert), exchange(send_src)
    by_expert = torch.argsort(expert.to(torch.int64), stable=True)              # receiver: group by local expert
    return {"rows": rows[by_expert], "src": src[by_expert],
            "count": torch.bincount(expert.to(torch.int64), minlength=epr).to(torch.int32)}
