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


# ---- the destination-agnostic layer across ranks ------------------------------------------------------
#
# One EpRank per GPU.  A layer step is five phases with a barrier between them (every rank's kernels of the
# phase complete before any rank starts the next): begin (own counters to their start state) -> dispatch
# (route the own tokens, push their rows into the owners' regions) -> experts (tile table from the own
# allocation pointers, expert FFN on the own regions) -> send_back (result rows to the source ranks' staging
# buffers) -> finish (weighted sum over each own token's K staged rows).  No rank ever tells another one counts
# or offsets; the only cross-rank traffic is the rows, the remote atomics and the counters.  The kernels wait
# for nobody, so the phases may also be run rank after rank on a single GPU (run_in_process, used by the
# tests) or by several processes sharing one GPU through CUDA IPC (EpGroup).
#
# Not measured on more than one GPU.

class EpRank:
    SHARED = ("recv", "row_pointer", "tile_count", "src_info", "rows_done", "staging", "rows_back")

    def __init__(self, rank: int, R: int, T_local: int, H: int, E: int, K: int, F: int, dtype: int,
                 cap_rows: int | None = None, device="cuda"):
        from . import binding as B
        self.B = B
        self.rank, self.R, self.T, self.H, self.E, self.K, self.F, self.dtype = rank, R, T_local, H, E, K, F, dtype
        self.epr = E // R
        # overflow-free capacity: an expert is picked at most once per token of the whole batch
        self.cap = cap_rows if cap_rows else (R * T_local + 127) // 128 * 128
        self.device = torch.device(device)
        el = torch.bfloat16 if dtype == B.DTYPE_BF16 else torch.float32
        self.el = el
        self.cfg = B.make_config(T_local, H, E, R, K, F, dtype)                       # what the peer kernels see
        # routing and the final weighted sum run on the rank's own tokens; the experts on its static regions
        self.token_plan = B.Plan(B.make_config(T_local, H, E, R, K, 0, dtype, identity_experts=1), device=device)
        self.expert_plan = B.Plan(B.make_config(128, H, self.epr, 1, 1, F, dtype, dispatch_mode=B.DISPATCH_ATOMIC_STATIC,
                                                capacity_rows=self.cap), device=device)
        d = self.device
        self.own = make_receive_buffers(E, R, H, self.cap, el, d)
        self.own["staging"] = torch.zeros((T_local * K, H), dtype=el, device=d)
        self.own["rows_back"] = torch.zeros(1, dtype=torch.int32, device=d)
        self.out_rows = torch.empty((self.epr * self.cap, H), dtype=el, device=d)
        self.expert_count = torch.zeros(self.epr, dtype=torch.int32, device=d)
        self.tile_expert = torch.full((self.epr * self.cap // 128,), -1, dtype=torch.int32, device=d)
        self.topk_idx = torch.empty((T_local, K), dtype=torch.int32, device=d)
        self.topk_w = torch.empty((T_local, K), dtype=torch.float32, device=d)
        self.slot_of = torch.empty((T_local, K), dtype=torch.int32, device=d)
        self.status = torch.zeros(4, dtype=torch.int32, device=d)
        self.peers = None

    def connect(self, peers: list[dict]) -> None:
        """peers[r]: rank r's SHARED buffers as tensors or device pointers valid on this GPU (own entry included)."""
        if len(peers) != self.R:
            raise ValueError("one entry per rank")
        self.peers = peers

    # ---- phases -------------------------------------------------------------------------------------
    def begin(self) -> None:
        for k in ("row_pointer", "tile_count", "rows_done", "rows_back"):
            self.own[k].zero_()
        self.own["src_info"].fill_(-1)

    def dispatch(self, x, wr, bias) -> None:
        self.token_plan.moe_route(x, wr, bias, self.topk_idx, self.topk_w)
        self.B.moe_dispatch_ep(self.cfg, self.rank, self.peers, self.cap, x, self.topk_idx, self.slot_of, self.status[:2])

    def experts(self, wg, wu, wd) -> None:
        """wg, wu [E/R, F, H], wd [E/R, H, F]: this rank's experts."""
        self.B.moe_ep_tiles(self.epr, self.cap, self.own["row_pointer"], self.expert_count, self.tile_expert)
        self.expert_plan.moe_expert_ffn(self.own["recv"], self.tile_expert, wg, wu, wd, self.out_rows, None, None)

    def send_back(self) -> None:
        self.B.moe_combine_ep(self.cfg, [q["staging"] for q in self.peers], [q["rows_back"] for q in self.peers], self.cap,
                              self.out_rows, self.own["src_info"], self.expert_count, self.status[2:])

    def finish(self, y) -> None:
        self.token_plan.moe_combine_staged(self.own["staging"], self.slot_of, self.topk_w, y)
        torch.cuda.synchronize(self.device)
        st = self.status.tolist()
        if st[0] or st[2]:
            raise self.B.MoeError(st[0] or st[2], f"expert-parallel step on rank {self.rank} (detail {st[1] or st[3]})")
        code, detail = self.expert_plan.moe_last_status()
        if code:
            raise self.B.MoeError(code, f"expert kernel on rank {self.rank} (detail {detail})")


def run_in_process(ranks: list[EpRank], xs, wr, bias, wgs, wus, wds, ys) -> None:
    """All ranks in one process on one GPU, phase by phase (the peers' buffers are plain local memory)."""
    for r in ranks:
        r.connect([q.own for q in ranks])
    for r in ranks:
        r.begin()
    for r, x in zip(ranks, xs):
        r.dispatch(x, wr, bias)
    for r, wg, wu, wd in zip(ranks, wgs, wus, wds):
        r.experts(wg, wu, wd)
    for r in ranks:
        r.send_back()
    for r, y in zip(ranks, ys):
        r.finish(y)


class EpGroup:
    """One EpRank per process: exchanges CUDA IPC handles of the shared buffers over a torch.distributed group
    (any backend that can all_gather_object: gloo is enough) and runs the phases with barriers in between."""

    def __init__(self, rank_obj: EpRank, group=None):
        from torch.multiprocessing.reductions import reduce_tensor
        self.r, self.group = rank_obj, group
        me = dist.get_rank(group)
        if me != rank_obj.rank or dist.get_world_size(group) != rank_obj.R:
            raise ValueError("the process group's rank and size must be the layer's")
        mine = {k: reduce_tensor(rank_obj.own[k]) for k in EpRank.SHARED}
        everyone = [None] * rank_obj.R
        dist.all_gather_object(everyone, mine, group=group)
        self.keep = []          # the mapped tensors keep the IPC mappings open
        peers = []
        for r, handles in enumerate(everyone):
            if r == me:
                peers.append(rank_obj.own)
                continue
            mapped = {k: fn(*args) for k, (fn, args) in handles.items()}
            self.keep.append(mapped)
            for t in mapped.values():
                if t.device != rank_obj.device:
                    # Another GPU's memory: a small copy makes torch enable peer access between the two devices,
                    # which the kernels' plain loads and stores need as well.
                    t.view(-1)[:1].to(rank_obj.device)
                    break
            peers.append({k: t.data_ptr() for k, t in mapped.items()})
        rank_obj.connect(peers)
        self.barrier()

    def barrier(self) -> None:
        torch.cuda.synchronize(self.r.device)
        dist.barrier(group=self.group)

    def step(self, x, wr, bias, wg, wu, wd, y) -> None:
        r = self.r
        r.begin()
        self.barrier()
        r.dispatch(x, wr, bias)
        self.barrier()
        r.experts(wg, wu, wd)
        r.send_back()
        self.barrier()
        r.finish(y)

    def close(self) -> None:
        self.barrier()          # nobody still writes into a buffer that is about to go away
        self.keep.clear()
