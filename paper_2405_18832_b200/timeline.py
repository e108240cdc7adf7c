"""Per-unit device timeline of the expert FFN kernel, summarised per segment of the unit list.

    python -m paper_2405_18832_b200.timeline C1 [C2 C3 HOTPROBE ...] [--pairs]

Runs the layer a few times on cuda:0 with the L2 flushed, switches the kernel's timeline on for
one call (monde_diag_set_trace: every CTA records, per unit it ran, the unit id, the producer's
first and last load issue, the first operands ready, the accumulator commit, the epilogue's start
and end and the time the MMA issuer spent waiting for operands, all on the global nanosecond
timer) and prints, per segment of the list (hot / cold, first / second layer): units, mean times,
when the segment started and ended, and how many CTAs were in which segment every 5 us.

A measurement aid: nothing here computes anything of the layer.  Segment boundaries are worked out
from the routing result with the kernel's own rules (token tile 256 for hot experts, threshold - 1
rounded up to 16 and at most 64 for cold ones; two feature tiles per unit for the cold class and,
from d_model 1536 on, for the hot class).
"""
from __future__ import annotations

import ctypes
import sys

import numpy as np
import torch

from . import binding as B
from . import synthetic as S

SLOTS = 128          # units recorded per CTA
FIELDS = ("unit", "issue_first", "issue_last", "operands_first", "commit", "epilogue_start", "epilogue_end", "waited_ns")
SEGMENTS = ("hot L1", "hot L2", "cold L1", "cold L2")


def record(name: str, pairs: bool = False):
    """One traced FFN call of workload `name`; returns (problem, counts, cls, trace[sms, SLOTS, 8])."""
    w = S.config(name)
    p = w.problem
    g = S.generate(w, with_weights=False)
    g.update({k: v for k, v in S.generate(w, weights_device="cuda").items() if k in ("W1", "W2", "b1", "b2")})
    d = {k: (None if v is None else v.cuda()) for k, v in g.items()}
    buf = B.LayerBuffers(p)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    trace = torch.zeros(sms * SLOTS * 8, dtype=torch.int64, device="cuda")
    L = B.lib()
    L.monde_diag_set_ffn_cta_pairs(1 if pairs else -1)
    try:
        for i in range(4):
            flush.fill_(i)
            if i == 3:
                L.monde_diag_set_trace(ctypes.c_void_p(trace.data_ptr()), SLOTS)
            B.moe_ffn_layer_forward(p, d["x"], d["Wg"], d["bg"], d["W1"], d["b1"], d["W2"], d["b2"], buf)
        B.monde_poll_device_status(buf.ws)
    finally:
        L.monde_diag_set_trace(ctypes.c_void_p(0), 0)
        L.monde_diag_set_ffn_cta_pairs(-1)
    return p, buf.counts.cpu().numpy(), buf.cls.cpu().numpy(), trace.cpu().numpy().reshape(sms, SLOTS, 8)


def segment_bounds(p, counts, cls, pairs: bool = False):
    """Ends of the first three segments of the unit list (the fourth runs to the end)."""
    wide = p.d_model >= 1536 or pairs
    tpu_hot = 2 if wide else 1
    cold_tile = min(64, max(16, (p.hot_threshold - 1 + 15) // 16 * 16))
    tt_hot = sum(max(1, -(-int(m) // 256)) for m, c in zip(counts, cls) if c == 2)
    tt_cold = sum(max(1, -(-int(m) // cold_tile)) for m, c in zip(counts, cls) if c == 1)
    nt1, nt2 = -(-p.d_ff // 128), -(-p.d_model // 128)
    seg1 = tt_hot * -(-nt1 // tpu_hot)
    seg2 = seg1 + tt_hot * -(-nt2 // tpu_hot)
    seg3 = seg2 + tt_cold * -(-nt1 // 2)
    return seg1, seg2, seg3


def summarise(name: str, pairs: bool = False, out=sys.stdout) -> None:
    p, counts, cls, t = record(name, pairs)
    seg1, seg2, seg3 = segment_bounds(p, counts, cls, pairs)
    valid = t[:, :, 6] > 0
    if pairs:
        valid &= t[:, :, 4] > 0           # the CTA of a pair that issues the MMAs
    if not valid.any():
        print(f"{name}: nothing recorded", file=out)
        return
    t0 = t[:, :, 1][valid].min()
    us = lambda a: a / 1e3
    ids = t[:, :, 0]
    seg = np.where(ids < seg1, 0, np.where(ids < seg2, 1, np.where(ids < seg3, 2, 3)))
    print(f"{name}: {int(valid.sum())} units on {int(valid.any(axis=1).sum())} CTAs; list segments end at {seg1}, {seg2}, {seg3}", file=out)
    for s_, label in enumerate(SEGMENTS):
        m = valid & (seg == s_)
        if not m.any():
            continue
        issue = us(t[:, :, 2] - t[:, :, 1])[m]
        span = us(t[:, :, 4] - t[:, :, 3])[m]
        epi = us(t[:, :, 6] - t[:, :, 5])[m]
        wait = us(t[:, :, 7])[m]
        print(f"  {label:7s} units {int(m.sum()):5d}  loads first->last {issue.mean():6.2f}  operands->commit {span.mean():6.2f} "
              f"(waiting {wait.mean():5.2f})  epilogue {epi.mean():5.2f}  | first load at {us(t[:, :, 1][m].min() - t0):6.1f}, "
              f"last epilogue end {us(t[:, :, 6][m].max() - t0):6.1f} us", file=out)
    ends = np.array([us(t[c, :, 6][valid[c]].max() - t0) for c in range(t.shape[0]) if valid[c].any()])
    per_cta = valid.sum(axis=1)
    print(f"  CTAs end between {ends.min():.1f} and {ends.max():.1f} us (median {np.median(ends):.1f}); units per CTA "
          f"{int(per_cta[per_cta > 0].min())}-{int(per_cta.max())}", file=out)
    step = 5 if ends.max() < 400 else 50
    for at in range(0, int(ends.max()) + step, step):
        row = [int((valid & (seg == s_) & (us(t[:, :, 1] - t0) <= at) & (us(t[:, :, 6] - t0) >= at)).any(axis=1).sum())
               for s_ in range(4)]
        print(f"  t = {at:4d} us  CTAs in {' / '.join(SEGMENTS)}: {row}", file=out)


if __name__ == "__main__":
    args = [a for a in sys.argv[1:] if not a.startswith("--")]
    for n in args or ["C1"]:
        summarise(n, pairs="--pairs" in sys.argv)
