"""Expert FFN of one MoE layer split over several GPUs by expert (one process per GPU).

Paper, Section 3.3, last paragraph: with several devices the experts' workloads are sorted by
compute intensity and dealt out round-robin, every device receives the input activations of the
experts dealt to it, computes them, and the outputs come back for the combine.  On B200s the
cost of an expert is streaming its weights from HBM, so dealing the activated experts over G
GPUs divides the weight bytes each GPU streams by about G; the price is one exchange of routed
rows out and one back.

Reading of the paper used here (it does not say where the parameters live when the deal changes
from batch to batch): every rank holds all expert weights (8.6 GB for the NLLB-like layer against
180 GB of HBM) and a batch of its own tokens.  Per layer call, on every rank:

  1. route and permute the rank's own tokens (monde_route, monde_permute: unchanged);
  2. all-gather the per-expert counts (E integers per rank), add them up, deal the experts:
     sorted by total count (most tokens first, equal counts: smaller id first), expert number i of
     that order goes to rank i mod G - the same result on every rank, no negotiation;
  3. send each expert's rows of x_perm to its owner (one all-to-all with per-rank row counts);
     the owner lays the received rows out expert-contiguously (expert ascending, source rank
     ascending) and runs the expert FFN on them with the summed counts of the experts it owns;
  4. send the output rows back the same way; every rank finds y_perm in its own row order and
     combines as usual.

The exchange is torch.distributed all_to_all_single (NCCL over NVLink on GPUs, gloo on CPUs);
received rows land in this GPU's memory before any kernel reads them, and no kernel is handed
another GPU's memory.  This module only builds index lists and moves rows; the arithmetic is the
`ffn` callable (on GPUs: monde_moe_ffn_fwd through `binding_ffn`).

Status: the bookkeeping is tested with two gloo ranks on CPUs against the single-device result and
the owner-side GPU path with a process group of one NCCL rank; it has not run on more than one GPU.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, Optional

import torch
import torch.distributed as dist


def deal_experts(total_counts: torch.Tensor, world: int) -> torch.Tensor:
    """owner[e] for every expert: experts in order of decreasing total count (equal counts: smaller id
    first) are dealt to ranks 0, 1, ..., world-1, 0, 1, ...  Experts without tokens are dealt too (they
    cost nothing).  Pure function of the counts, so every rank computes the same deal."""
    c = total_counts.to(torch.int64).cpu()
    E = c.numel()
    order = torch.argsort(-c * E + torch.arange(E, dtype=torch.int64), stable=True)
    # key (-count, id) ascending == count descending, id ascending; exact in int64
    owner = torch.empty(E, dtype=torch.int64)
    owner[order] = torch.arange(E, dtype=torch.int64) % world
    return owner


@dataclass
class ExchangePlan:
    """Index lists of one layer call on one rank (all on the CPU; tiny)."""
    owner: torch.Tensor           # [E] rank that computes each expert
    send_index: torch.Tensor      # rows of the local x_perm in the order they are sent (by owner, then expert id)
    send_splits: list             # rows sent to each rank
    recv_splits: list             # rows received from each rank
    regroup_index: torch.Tensor   # received rows -> expert-contiguous order (expert ascending, source rank ascending)
    local_counts: torch.Tensor    # [E] rows this rank computes for each expert (0 for experts it does not own)
    local_offsets: torch.Tensor   # [E+1] exclusive scan of local_counts


def build_plan(all_counts: torch.Tensor, rank: int) -> ExchangePlan:
    """`all_counts` [world, E]: every rank's per-expert assignment counts (the all-gathered histograms)."""
    all_counts = all_counts.to(torch.int64).cpu()
    world, E = all_counts.shape
    owner = deal_experts(all_counts.sum(0), world)
    mine = all_counts[rank]
    my_offsets = torch.zeros(E + 1, dtype=torch.int64)
    my_offsets[1:] = torch.cumsum(mine, 0)
    # rows leave grouped by destination, experts ascending inside a destination
    send_chunks, send_splits = [], []
    for dst in range(world):
        n = 0
        for e in torch.nonzero(owner == dst).flatten().tolist():
            if mine[e] > 0:
                send_chunks.append(torch.arange(my_offsets[e], my_offsets[e + 1]))
                n += int(mine[e])
        send_splits.append(n)
    send_index = torch.cat(send_chunks) if send_chunks else torch.zeros(0, dtype=torch.int64)
    # rows arrive grouped by source, experts ascending inside a source; position of (src, e) in that stream:
    owned = torch.nonzero(owner == rank).flatten().tolist()
    recv_splits = [int(all_counts[src, owned].sum()) if owned else 0 for src in range(world)]
    start = {}
    pos = 0
    for src in range(world):
        for e in owned:
            start[(src, e)] = pos
            pos += int(all_counts[src, e])
    regroup, local_counts = [], torch.zeros(E, dtype=torch.int64)
    for e in owned:
        for src in range(world):
            n = int(all_counts[src, e])
            if n:
                regroup.append(torch.arange(start[(src, e)], start[(src, e)] + n))
            local_counts[e] += n
    regroup_index = torch.cat(regroup) if regroup else torch.zeros(0, dtype=torch.int64)
    local_offsets = torch.zeros(E + 1, dtype=torch.int64)
    local_offsets[1:] = torch.cumsum(local_counts, 0)
    return ExchangePlan(owner, send_index, send_splits, recv_splits, regroup_index, local_counts, local_offsets)


def _wire(t: torch.Tensor) -> torch.Tensor:
    """Rows as plain bytes: every backend moves those (16-bit types are not universal)."""
    return t.view(torch.uint8)


def _all_to_all_rows(rows: torch.Tensor, send_splits, recv_splits, group) -> torch.Tensor:
    rows = rows.contiguous()
    out = torch.empty((sum(recv_splits),) + tuple(rows.shape[1:]), dtype=rows.dtype, device=rows.device)
    dist.all_to_all_single(_wire(out), _wire(rows), output_split_sizes=list(recv_splits),
                           input_split_sizes=list(send_splits), group=group)
    return out


FfnFn = Callable[[torch.Tensor, torch.Tensor, torch.Tensor], torch.Tensor]


def expert_parallel_ffn(x_perm: torch.Tensor, counts: torch.Tensor, ffn: FfnFn,
                        group: Optional[dist.ProcessGroup] = None) -> torch.Tensor:
    """Steps 2-4 of the module docstring.  `x_perm` [A, d_model]: this rank's routed rows in
    expert-contiguous order; `counts` [E]: this rank's histogram.  `ffn(rows, local_counts, local_offsets)`
    computes the expert FFN of expert-contiguous rows (rows of expert e at local_offsets[e] ..) and
    returns the output rows in the same order.  Returns y_perm [A, d_model] in this rank's row order."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    mine = counts.to(torch.int64).to(x_perm.device)
    gathered = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine, group=group)
    plan = build_plan(torch.stack([g.cpu() for g in gathered]), rank)
    dev = x_perm.device
    send_index = plan.send_index.to(dev)
    regroup = plan.regroup_index.to(dev)
    received = _all_to_all_rows(x_perm.index_select(0, send_index), plan.send_splits, plan.recv_splits, group)
    x_local = received.index_select(0, regroup)                      # expert-contiguous on the owner
    y_local = ffn(x_local, plan.local_counts, plan.local_offsets)
    back = torch.empty_like(y_local)
    back[regroup] = y_local                                          # the order the rows arrived in
    returned = _all_to_all_rows(back, plan.recv_splits, plan.send_splits, group)
    y_perm = torch.empty((x_perm.shape[0],) + tuple(returned.shape[1:]), dtype=returned.dtype, device=dev)
    y_perm[send_index] = returned                                    # this rank's own row order
    return y_perm


def binding_ffn(p, W1, b1, W2, b2, stream=None) -> FfnFn:
    """The `ffn` callable for GPUs: monde_moe_ffn_fwd on the rows a rank received, with the threshold
    classes of the summed counts.  Problem `p` describes one rank's batch (T tokens, top_k); a rank may
    receive up to world * T * top_k rows, so buffers are sized per call."""
    import dataclasses

    from . import binding as B

    def run(rows, local_counts, local_offsets):
        dev = rows.device
        n = rows.shape[0]
        E = local_counts.numel()
        # the received rows are described to the library as a top-1 problem of n tokens
        q = dataclasses.replace(p, T=max(n, 1), top_k=1)
        counts = local_counts.to(torch.int32).to(dev)
        offsets = local_offsets.to(torch.int32).to(dev)
        active = local_counts > 0
        hot = active & (local_counts >= p.hot_threshold)
        cls = (active.to(torch.uint8) + hot.to(torch.uint8)).to(dev)
        hot_ids = torch.full((E,), -1, dtype=torch.int32)
        cold_ids = torch.full((E,), -1, dtype=torch.int32)
        hi = torch.nonzero(hot).flatten().to(torch.int32)
        ci = torch.nonzero(active & ~hot).flatten().to(torch.int32)
        hot_ids[: hi.numel()] = hi
        cold_ids[: ci.numel()] = ci
        n_hot_cold = torch.tensor([hi.numel(), ci.numel()], dtype=torch.int32, device=dev)
        y = torch.empty_like(rows)
        if n == 0:
            return y
        ws = torch.zeros(B.monde_workspace_bytes(q), dtype=torch.uint8, device=dev)
        B.monde_moe_ffn_fwd(q, rows, W1, b1, W2, b2, counts, offsets, cls, hot_ids.to(dev), cold_ids.to(dev),
                            n_hot_cold, y, ws, stream)
        return y

    return run
