"""The paper's GPU-MoNDE load-balancing policy on one GPU (Section 3.3, Eq. 3-6).

`monde_classify_top_h` (in the CUDA library) picks the hot experts as the H experts with the most
tokens, H = floor(alpha * BW_a / (BW_b + BW_a) * Expert_Activ).  This module holds the host-side
part: the inverse of Eq. 6 and the paper's auto-tuner for alpha, which replays a few recent
batches with H and its neighbours (the paper names H+1 and H+2 as examples of candidates) and keeps
the fastest, i.e. walks to a local optimum over repeated tuning rounds (Section 3.3, last paragraph).  On one
B200 both classes read weights from HBM, so BW_a and BW_b are the effective weight-streaming rates
of the two tilings; their ratio only sets the starting point that alpha then corrects.
"""
from __future__ import annotations

import math
from typing import Iterable, Sequence, Tuple

import torch

from . import binding as B


def h_of(alpha: float, active: int, bw_hot_feed: float, bw_cold_feed: float) -> int:
    """Eq. 6, rounded down and clamped to [0, active]."""
    h = alpha * bw_hot_feed / (bw_cold_feed + bw_hot_feed) * active
    return max(0, min(active, int(math.floor(h)) if h > 0 else 0))


def alpha_for_h(h: int, active: int, bw_hot_feed: float, bw_cold_feed: float) -> float:
    """An alpha that makes Eq. 6 give exactly `h` hot experts for `active` activated experts
    (the middle of the interval of such alphas)."""
    share = bw_hot_feed / (bw_cold_feed + bw_hot_feed)
    return (h + 0.5) / (share * max(active, 1))


def autotune_alpha(p, batches: Iterable[torch.Tensor], Wg, bg, W1, b1, W2, b2, alpha: float,
                   bw_hot_feed: float, bw_cold_feed: float, candidates: Sequence[int] = (-2, -1, 0, 1, 2),
                   reps: int = 3) -> Tuple[float, dict]:
    """One tuning round: replays `batches` (device tensors [T, d_model]) with H + c hot experts for
    every c in `candidates`, H from the current alpha, and returns (new alpha, report).  The expert
    FFN call is what is timed (CUDA events); routing and permutation do not depend on the classes.
    The default candidates look both ways, since on one GPU too many hot experts cost time as well
    as too few; pass (0, 1, 2) for the upward-only search of the paper's example."""
    buf = B.LayerBuffers(p)
    stream = torch.cuda.current_stream()
    total_ms = {c: 0.0 for c in candidates}
    actives = []
    for x in batches:
        B.monde_route(p, x, Wg, bg, buf.topk_idx, buf.topk_w, buf.counts, buf.offsets, buf.cls, buf.hot_ids,
                      buf.cold_ids, buf.n_hot_cold, None, buf.ws)
        B.monde_permute(p, x, buf.topk_idx, buf.offsets, buf.perm, buf.inv_perm, buf.x_perm, buf.ws)
        active = int((buf.counts > 0).sum().item())
        actives.append(active)
        h0 = h_of(alpha, active, bw_hot_feed, bw_cold_feed)
        for c in candidates:
            a_c = alpha_for_h(max(0, min(active, h0 + c)), active, bw_hot_feed, bw_cold_feed)
            B.monde_classify_top_h(p, buf.counts, a_c, bw_hot_feed, bw_cold_feed, buf.cls, buf.hot_ids,
                                   buf.cold_ids, buf.n_hot_cold)
            best = float("inf")
            for _ in range(reps + 1):          # first run is a warm-up
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                B.monde_moe_ffn_fwd(p, buf.x_perm, W1, b1, W2, b2, buf.counts, buf.offsets, buf.cls, buf.hot_ids,
                                    buf.cold_ids, buf.n_hot_cold, buf.y_perm, buf.ws)
                e1.record(stream)
                e1.synchronize()
                best = min(best, e0.elapsed_time(e1))
            total_ms[c] += best
    B.monde_poll_device_status(buf.ws)
    best_c = min(candidates, key=lambda c: total_ms[c])
    mean_active = sum(actives) / max(len(actives), 1)
    h_mean = h_of(alpha, int(round(mean_active)), bw_hot_feed, bw_cold_feed)
    h_new = max(0, min(int(round(mean_active)), h_mean + best_c))
    new_alpha = alpha if best_c == 0 else alpha_for_h(h_new, int(round(mean_active)), bw_hot_feed, bw_cold_feed)
    return new_alpha, {"ms": total_ms, "chosen_offset": best_c, "mean_active": mean_active, "h_before": h_mean,
                       "h_after": h_new if best_c != 0 else h_mean}


def autotune_alpha_rounds(p, batches, Wg, bg, W1, b1, W2, b2, alpha: float, bw_hot_feed: float,
                          bw_cold_feed: float, rounds: int = 4, **kw) -> Tuple[float, list]:
    """The periodic re-tuning of Section 3.3 run `rounds` times on the same replayed batches; stops
    early at a local optimum (a round that keeps H).  Returns (alpha, list of per-round reports)."""
    batches = list(batches)
    reports = []
    for _ in range(rounds):
        alpha, rep = autotune_alpha(p, batches, Wg, bg, W1, b1, W2, b2, alpha, bw_hot_feed, bw_cold_feed, **kw)
        reports.append(rep)
        if rep["chosen_offset"] == 0:
            break
    return alpha, reports
