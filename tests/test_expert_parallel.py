"""Expert-parallel split of the expert FFN (paper Section 3.3, multi-device paragraph): the deal of
experts to ranks and the two exchanges, run as two gloo ranks on CPUs.  Every rank routes its own
tokens with the oracle, sends each expert's rows to the rank the expert was dealt to, computes what it
received with the oracle's expert FFN, sends the outputs back and combines; the result must be what
the oracle gives for that rank's tokens on one device, exactly (same rows, same arithmetic per row)."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from paper_2405_18832_b200 import expert_parallel as EP

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_deal_is_round_robin_in_order_of_count():
    counts = torch.tensor([5, 0, 9, 9, 1, 0, 7, 3])
    owner = EP.deal_experts(counts, 3)
    # order by count (ties: smaller id): 2, 3, 6, 0, 7, 4, 1, 5 -> ranks 0, 1, 2, 0, 1, 2, 0, 1
    assert owner.tolist() == [0, 0, 0, 1, 2, 1, 2, 1]
    for world in (1, 2, 4, 8):
        big = torch.arange(64) ** 2 % 37
        own = EP.deal_experts(big, world)
        load = [int(big[own == r].sum()) for r in range(world)]
        per = [int((own == r).sum()) for r in range(world)]
        assert max(per) - min(per) <= 1                       # experts spread evenly
        assert max(load) - min(load) <= int(big.max())        # and so is the work, to within one expert


def test_plan_row_bookkeeping_is_consistent():
    rng = np.random.default_rng(3)
    all_counts = torch.from_numpy(rng.integers(0, 6, size=(3, 10)))
    plans = [EP.build_plan(all_counts, r) for r in range(3)]
    for r, pl in enumerate(plans):
        assert sorted(pl.send_index.tolist()) == list(range(int(all_counts[r].sum())))      # every row leaves once
        assert sum(pl.recv_splits) == int(pl.local_counts.sum()) == pl.regroup_index.numel()
        assert sorted(pl.regroup_index.tolist()) == list(range(sum(pl.recv_splits)))
        assert pl.local_counts.tolist() == [int(all_counts[:, e].sum()) if pl.owner[e] == r else 0 for e in range(10)]
        for dst in range(3):
            assert pl.send_splits[dst] == plans[dst].recv_splits[r]                          # both ends agree
    assert int(sum(p.local_counts.sum() for p in plans)) == int(all_counts.sum())


RANK_SCRIPT = r"""
import json, os, sys
sys.path.insert(0, {root!r})
import numpy as np, torch, torch.distributed as dist
import oracle
from paper_2405_18832_b200 import expert_parallel as EP, synthetic as S
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
w = S.Workload("ep", S.Problem(96, 64, 128, 12, 2, 8, 1, {dtype!r}, "gelu"), 1.2, 40 + rank, "random")
g = S.generate(w)
shared = S.generate(S.Workload("ep", w.problem, 1.2, 40, "random"))      # one set of gate / expert weights for all ranks
for k in ("Wg", "bg", "W1", "b1", "W2", "b2"):
    g[k] = shared[k]
h = {{k: S.as_numpy(v) for k, v in g.items()}}
p = w.problem
single = oracle.moe_layer(h["x"], h["Wg"], h["bg"], h["W1"], h["b1"], h["W2"], h["b2"], p.top_k, p.renormalize,
                          p.hot_threshold, p.act)
r = single.route
x_perm = torch.from_numpy(single.perm.x_perm.copy())
if {dtype!r} == "bf16":
    x_perm = x_perm.view(torch.int16).view(torch.bfloat16)
seen = {{}}
def ffn(rows, local_counts, local_offsets):
    seen["counts"] = local_counts.tolist()
    rows_np = S.as_numpy(rows)
    experts = oracle.experts_of_rows(local_offsets.numpy().astype(np.int32))
    y = oracle.expert_ffn(rows_np, experts, h["W1"], h["b1"], h["W2"], h["b2"], p.act)
    return torch.from_numpy(y)                                            # fp64 rows travel back
y_perm = EP.expert_parallel_ffn(x_perm, torch.from_numpy(r.counts), ffn)
out = oracle.combine(y_perm.numpy(), single.perm.inv_perm, r.topk_w)
owned = [e for e, c in enumerate(seen["counts"]) if c > 0]
print(json.dumps(dict(rank=rank, equal_y=bool(np.array_equal(y_perm.numpy(), single.y_perm)),
                      equal_out=bool(np.array_equal(out, single.out)), rows_in=int(sum(seen["counts"])),
                      rows_mine=int(r.counts.sum()), owned=owned, counts=r.counts.tolist())))
dist.barrier()
dist.destroy_process_group()
"""


def _run_two_ranks(tmp_path, dtype, port):
    script = tmp_path / "rank.py"
    script.write_text(RANK_SCRIPT.format(root=ROOT, dtype=dtype))
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, text=True))
    outs = [json.loads(p.communicate(timeout=300)[0].strip().splitlines()[-1]) for p in procs]
    assert all(p.returncode == 0 for p in procs)
    return sorted(outs, key=lambda o: o["rank"])


def test_two_ranks_reproduce_the_single_device_layer(tmp_path):
    for dtype, port in (("bf16", 29551), ("f32", 29552)):
        a, b = _run_two_ranks(tmp_path, dtype, port)
        assert a["equal_y"] and b["equal_y"] and a["equal_out"] and b["equal_out"]
        assert not set(a["owned"]) & set(b["owned"])                     # an expert is computed on one rank only
        total = np.array(a["counts"]) + np.array(b["counts"])
        assert set(a["owned"]) | set(b["owned"]) == {e for e in range(12) if total[e] > 0}
        assert a["rows_in"] + b["rows_in"] == a["rows_mine"] + b["rows_mine"] == 2 * 96 * 2
        # the deal: experts in order of total count alternate between the ranks
        order = sorted(range(12), key=lambda e: (-total[e], e))
        expect_a = {e for i, e in enumerate(order) if i % 2 == 0 and total[e] > 0}
        assert set(a["owned"]) == expect_a


@pytest.mark.gpu
def test_owner_side_ffn_on_the_gpu_gives_the_bytes_of_the_single_device_call():
    # One rank, one GPU (NCCL process group of size 1): every expert is dealt to this rank and the two exchanges
    # send the rows to itself, so what is exercised is the GPU side of the split - rows gathered in send order,
    # regrouped, described to the library as a top-1 problem of n rows with the summed counts, sent back and
    # scattered - against monde_moe_ffn_fwd called directly on the same routed rows.  More ranks than one need
    # more GPUs than this machine gives a test.
    import torch.distributed as dist

    import parity as P
    from paper_2405_18832_b200 import binding as B
    from paper_2405_18832_b200 import synthetic as S
    w = S.Workload("ep_gpu", S.Problem(700, 256, 512, 16, 2, 24, 1, "bf16", "gelu"), 1.2, 7, "random")
    p = w.problem
    dev = P.to_device(S.generate(w))
    buf = P.run_gpu(p, dev, want_probs=False)           # route, permute, FFN, combine on one device
    own = not dist.is_initialized()
    if own:
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29561", world_size=1, rank=0,
                                device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        ffn = EP.binding_ffn(p, dev["W1"], dev["b1"], dev["W2"], dev["b2"])
        y = EP.expert_parallel_ffn(buf.x_perm, buf.counts, ffn)
        torch.cuda.synchronize()
    finally:
        if own:
            dist.destroy_process_group()
    assert torch.equal(y, buf.y_perm)
