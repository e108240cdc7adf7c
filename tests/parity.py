"""Parity harness: runs the CUDA library through its binding and the CPU oracle on the
same seeded inputs and compares step by step.

Rules: routing integers, class lists, permutation and x_perm are bit-exact; gate
weights and probabilities agree to 1e-5 absolute (fp32 softmax); y_perm and out agree
within max|diff| <= 1e-2 * max|ref| and relative Frobenius error <= 5e-3 for bf16
problems, and within 1e-5 on both measures for fp32 problems.
"""
from __future__ import annotations

from types import SimpleNamespace

import numpy as np
import torch

import oracle
from paper_2405_18832_b200 import binding as B
from paper_2405_18832_b200 import synthetic as S

TOL = {"bf16": (1e-2, 5e-3), "f32": (1e-5, 1e-5)}


def widen(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def check_close(name, got64: np.ndarray, ref64: np.ndarray, dtype: str):
    tol_abs, tol_fro = TOL[dtype]
    if ref64.size == 0:
        return 0.0, 0.0
    scale = np.abs(ref64).max()
    max_abs = np.abs(got64 - ref64).max()
    fro = np.linalg.norm(got64 - ref64) / max(np.linalg.norm(ref64), 1e-300)
    assert np.isfinite(got64).all(), f"{name}: non-finite values"
    assert max_abs <= tol_abs * scale, f"{name}: max|diff| {max_abs:.3e} > {tol_abs:g} * {scale:.3e}"
    assert fro <= tol_fro, f"{name}: relative Frobenius error {fro:.3e} > {tol_fro:g}"
    return max_abs / max(scale, 1e-300), fro


def to_device(g, device="cuda"):
    return {k: (None if v is None else v.to(device)) for k, v in g.items()}


def run_gpu(p, dev, want_probs=True):
    buf = B.LayerBuffers(p, want_probs=want_probs)
    B.moe_ffn_layer_forward(p, dev["x"], dev["Wg"], dev["bg"], dev["W1"], dev["b1"], dev["W2"], dev["b2"], buf)
    B.monde_poll_device_status(buf.ws)
    return buf


def check_routing(p, g, buf):
    """Bit-exact integer outputs and 1e-5 gate weights against the oracle; returns the oracle's routing."""
    r = oracle.route(S.as_numpy(g["x"]), S.as_numpy(g["Wg"]), S.as_numpy(g["bg"]),
                     p.top_k, p.renormalize, p.hot_threshold)
    np.testing.assert_array_equal(buf.topk_idx.cpu().numpy(), r.topk_idx)
    np.testing.assert_array_equal(buf.counts.cpu().numpy(), r.counts)
    np.testing.assert_array_equal(buf.offsets.cpu().numpy(), r.offsets)
    np.testing.assert_array_equal(buf.cls.cpu().numpy(), r.cls)
    nh, nc = r.n_hot_cold
    np.testing.assert_array_equal(buf.n_hot_cold.cpu().numpy(), r.n_hot_cold)
    np.testing.assert_array_equal(buf.hot_ids.cpu().numpy()[:nh], r.hot_ids[:nh])
    np.testing.assert_array_equal(buf.cold_ids.cpu().numpy()[:nc], r.cold_ids[:nc])
    if p.T:
        assert np.abs(buf.topk_w.cpu().numpy().astype(np.float64) - r.topk_w).max() <= 1e-5
        if buf.probs is not None:
            assert np.abs(buf.probs.cpu().numpy().astype(np.float64) - r.probs).max() <= 1e-5
    pm = oracle.permute(S.as_numpy(g["x"]), r.topk_idx, r.offsets)
    np.testing.assert_array_equal(buf.perm.cpu().numpy(), pm.perm)
    np.testing.assert_array_equal(buf.inv_perm.cpu().numpy(), pm.inv_perm)
    np.testing.assert_array_equal(S.as_numpy(buf.x_perm), pm.x_perm)
    return r, pm


def check_full(w: S.Workload, g=None, dev=None):
    """Element-by-element parity of every output of the four calls."""
    p = w.problem
    g = g if g is not None else S.generate(w)
    dev = dev if dev is not None else to_device(g)
    buf = run_gpu(p, dev)
    r, pm = check_routing(p, g, buf)
    y_ref = oracle.expert_ffn(pm.x_perm, oracle.experts_of_rows(r.offsets), S.as_numpy(g["W1"]),
                              S.as_numpy(g["b1"]), S.as_numpy(g["W2"]), S.as_numpy(g["b2"]), p.act)
    y_err = check_close("y_perm", widen(buf.y_perm), y_ref, p.dtype)
    out_ref = oracle.combine(y_ref, pm.inv_perm, r.topk_w)
    out_err = check_close("out", widen(buf.out), out_ref, p.dtype)
    # combine checked alone: the oracle's combine applied to the device's own y_perm
    alone = oracle.combine(widen(buf.y_perm), pm.inv_perm, buf.topk_w.cpu().numpy().astype(np.float64))
    got = widen(buf.out)
    w64 = buf.topk_w.cpu().numpy().astype(np.float64)
    mag = oracle.combine(np.abs(widen(buf.y_perm)), pm.inv_perm, np.abs(w64))   # sum_j |w_j * y_j|
    ulp = 2.0 ** -8 if p.dtype == "bf16" else 2.0 ** -23
    bound = ulp * np.abs(alone) + p.top_k * 2.0 ** -23 * mag + 1e-30   # one output rounding + k fp32 steps
    assert (np.abs(got - alone) <= bound).all(), "combine: error beyond fp32 accumulation and one rounding"
    return SimpleNamespace(buf=buf, route=r, perm=pm, y_err=y_err, out_err=out_err)


class OracleSample:
    """Oracle outputs for a set of rows of the expert-contiguous buffer and a set of tokens, computed once
    and compared with any number of device runs on the same inputs (the expert outputs do not depend on
    the hot/cold classes).  Expert weights come to the host one expert at a time, so multi-gigabyte
    layers never need a host copy of all weights."""

    def __init__(self, w: S.Workload, g, dev, route, perm, rows=None, tokens=None):
        p = w.problem
        self.p, self.route, self.perm = p, route, perm
        A = p.T * p.top_k
        self.tokens = np.arange(p.T) if tokens is None else np.asarray(tokens, np.int64)
        need = perm.inv_perm[(self.tokens[:, None] * p.top_k + np.arange(p.top_k)[None, :]).reshape(-1)]
        rows = np.arange(A) if rows is None else np.asarray(rows, np.int64)
        self.rows = np.unique(np.concatenate([rows, need.astype(np.int64)]))
        row_expert = oracle.experts_of_rows(route.offsets)[self.rows]
        self.y_ref = np.zeros((self.rows.size, p.d_model))
        for e in np.unique(row_expert):          # one expert's weights on the host at a time
            sel = np.nonzero(row_expert == e)[0]
            W1 = S.as_numpy(dev["W1"][e:e + 1]); W2 = S.as_numpy(dev["W2"][e:e + 1])
            b1 = S.as_numpy(dev["b1"][e:e + 1]) if dev["b1"] is not None else None
            b2 = S.as_numpy(dev["b2"][e:e + 1]) if dev["b2"] is not None else None
            self.y_ref[sel] = oracle.expert_ffn(perm.x_perm[self.rows[sel]], np.zeros(sel.size, np.int32),
                                                W1, b1, W2, b2, p.act)
        # combine on the sampled tokens: their rows renumbered into the sample
        where = np.searchsorted(self.rows, need).astype(np.int32)
        self.out_ref = oracle.combine(self.y_ref, where, np.ascontiguousarray(route.topk_w[self.tokens]))
        self.experts_covered = np.unique(row_expert)

    def compare(self, buf, label=""):
        p = self.p
        y_got = widen(buf.y_perm[torch.as_tensor(self.rows, device=buf.y_perm.device)])
        y_err = check_close(f"y_perm{label}", y_got, self.y_ref, p.dtype)
        out_got = widen(buf.out[torch.as_tensor(self.tokens, device=buf.out.device)])
        out_err = check_close(f"out{label}", out_got, self.out_ref, p.dtype)
        assert torch.isfinite(buf.out.float()).all() and torch.isfinite(buf.y_perm.float()).all()
        return y_err, out_err


def sample_rows_by_expert(route, perm, p, n_tokens, row_budget):
    """Rows for a sampled comparison of a layer too large for the oracle in full: one whole expert
    from the few-token end of the histogram, one whole expert with at least 64 rows (hot at every
    threshold of the sweep), the rows around the first 256-row tile boundary of the busiest expert,
    and the rows of every (T / n_tokens)-th token."""
    counts, offsets = route.counts.astype(np.int64), route.offsets.astype(np.int64)
    active = np.nonzero(counts > 0)[0]
    rows = []
    least = active[np.argmin(counts[active])]
    rows.append(np.arange(offsets[least], offsets[least + 1]))
    big = active[counts[active] >= 64]
    if big.size:
        e = big[np.argmin(counts[big])]
        rows.append(np.arange(offsets[e], offsets[e + 1]))
    top = active[np.argmax(counts[active])]
    if counts[top] > 256:
        rows.append(offsets[top] + np.arange(224, min(counts[top], 304)))
    rows = np.unique(np.concatenate(rows))[:row_budget]
    tokens = np.arange(0, p.T, max(1, -(-p.T // n_tokens)))
    return rows, tokens


def check_by_expert(w: S.Workload, g, dev, thresholds=None, full_flop_limit=3.0e11, n_tokens=64, row_budget=512):
    """Parity of a layer whose weights live on the device only.  Routing integers are bit-exact in
    full at every threshold; expert outputs and the combined output are compared with the oracle on
    ALL rows and tokens when the layer is at most `full_flop_limit` flop, else on whole experts plus
    a token sample (sample_rows_by_expert).  Every threshold's device output is compared with the
    same oracle values."""
    import dataclasses
    p = w.problem
    thresholds = [p.hot_threshold] if thresholds is None else list(thresholds)
    sample, results = None, []
    for theta in thresholds:
        pt = dataclasses.replace(p, hot_threshold=theta)
        buf = run_gpu(pt, dev, want_probs=False)
        r, pm = check_routing(pt, g, buf)
        if sample is None:
            if 4.0 * p.A * p.d_model * p.d_ff <= full_flop_limit:
                sample = OracleSample(w, g, dev, r, pm)
            else:
                rows, tokens = sample_rows_by_expert(r, pm, p, n_tokens, row_budget)
                sample = OracleSample(w, g, dev, r, pm, rows, tokens)
        y_err, out_err = sample.compare(buf, f" theta={theta}")
        results.append(SimpleNamespace(buf=buf, route=r, perm=pm, y_err=y_err, out_err=out_err, theta=theta))
    return SimpleNamespace(sample=sample, runs=results, full=sample.rows.size == p.A)


def check_sampled(w: S.Workload, g, dev, n_tokens=96, buf=None):
    """Full-size parity: routing in full (bit-exact), expert outputs and the combined
    output on a deterministic sample of tokens, one oracle FFN row at a time."""
    p = w.problem
    buf = buf if buf is not None else run_gpu(p, dev, want_probs=False)
    r, pm = check_routing(p, g, buf)
    step = max(1, -(-p.T // n_tokens))
    tokens = np.arange(0, p.T, step)
    assign = (tokens[:, None] * p.top_k + np.arange(p.top_k)[None, :]).reshape(-1)
    rows = pm.inv_perm[assign]
    experts = r.topk_idx.reshape(-1)[assign]
    y_ref = np.zeros((rows.size, p.d_model))
    for e in np.unique(experts):          # one expert's weights on the host at a time
        sel = np.nonzero(experts == e)[0]
        W1 = S.as_numpy(dev["W1"][e:e + 1]); W2 = S.as_numpy(dev["W2"][e:e + 1])
        b1 = S.as_numpy(dev["b1"][e:e + 1]) if dev["b1"] is not None else None
        b2 = S.as_numpy(dev["b2"][e:e + 1]) if dev["b2"] is not None else None
        y_ref[sel] = oracle.expert_ffn(pm.x_perm[rows[sel]], np.zeros(sel.size, np.int32), W1, b1, W2, b2, p.act)
    y_got = widen(buf.y_perm[torch.as_tensor(rows, device=buf.y_perm.device).long()])
    y_err = check_close("y_perm(sample)", y_got, y_ref, p.dtype)
    out_ref = oracle.combine(y_ref, np.arange(rows.size, dtype=np.int32), np.ascontiguousarray(r.topk_w[tokens]))
    out_got = widen(buf.out[torch.as_tensor(tokens, device=buf.out.device).long()])
    out_err = check_close("out(sample)", out_got, out_ref, p.dtype)
    assert torch.isfinite(buf.out.float()).all() and torch.isfinite(buf.y_perm.float()).all()
    return SimpleNamespace(buf=buf, route=r, perm=pm, y_err=y_err, out_err=out_err, n_rows=rows.size)


GUARD_BYTES = 4096
GUARD_PATTERN = 0xA5


def guarded_layer_buffers(p):
    """LayerBuffers whose every output (and the workspace) sits between two guard regions filled with a
    pattern; returns (buf, check) where check() asserts that no guard byte changed.  Stands in for a
    memory checker: a store past either end of an output lands in a guard."""
    buf = B.LayerBuffers(p)
    guards = []
    for name in ("topk_idx", "topk_w", "counts", "offsets", "cls", "hot_ids", "cold_ids", "n_hot_cold", "perm",
                 "inv_perm", "x_perm", "y_perm", "out", "ws"):
        t = getattr(buf, name)
        nbytes = t.numel() * t.element_size()
        padded = (nbytes + 255) // 256 * 256              # keeps the rear guard off the tensor's last 16-byte vector
        raw = torch.full((GUARD_BYTES + padded + GUARD_BYTES,), GUARD_PATTERN, dtype=torch.uint8, device=t.device)
        body = raw[GUARD_BYTES:GUARD_BYTES + nbytes]
        if name == "ws":
            body.zero_()
        else:
            body.copy_(t.contiguous().view(-1).view(torch.uint8))   # keeps initial fills such as the -1 of the id lists
        setattr(buf, name, body.view(t.dtype).view(t.shape))
        guards.append((name, raw, nbytes))

    def check():
        torch.cuda.synchronize()
        for name, raw, nbytes in guards:
            front = raw[:GUARD_BYTES]
            rear = raw[GUARD_BYTES + nbytes:]
            assert bool((front == GUARD_PATTERN).all()), f"{name}: bytes before the buffer were written"
            assert bool((rear == GUARD_PATTERN).all()), f"{name}: bytes after the buffer were written"
    return buf, check
