"""The range-checking build of the library (libmonde_diag.so: the same sources with -DMONDE_DIAGNOSTICS).

It stands in for a memory checker: every index a kernel takes from memory is checked before it is used as
an address, violations are counted and the access is skipped.  Here: (1) ordinary layers run through it
without a single violation and give the bytes of the ordinary build; (2) inputs with indices out of range
(made on purpose, and only ever given to this build) are counted with the right site code while the guard
regions around every output stay untouched - nothing is written or read out of bounds, so nothing faults.
"""
import ctypes
import dataclasses

import pytest
import torch

import parity as P
from paper_2405_18832_b200 import binding as B
from paper_2405_18832_b200 import build as build_mod
from paper_2405_18832_b200 import synthetic as S

pytestmark = pytest.mark.gpu


def _violations():
    site, value = ctypes.c_int32(0), ctypes.c_longlong(0)
    n = B.lib().monde_diag_bounds_violations(ctypes.byref(site), ctypes.byref(value))
    return n, site.value, value.value


@pytest.fixture
def diag_lib(monkeypatch):
    path = build_mod.build(diagnostics=True)
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", path)
    assert _violations()[0] == 0
    yield
    assert B.lib().monde_diag_bounds_violations(None, None) >= 0      # still the checking build; record left clean


CASES = [
    S.Workload("diag_top2", S.Problem(333, 192, 448, 12, 2, 40, 1, "bf16", "gelu"), 1.0, 11, "random"),
    S.Workload("diag_wide", S.Problem(640, 1664, 1728, 6, 2, 100, 1, "bf16", "gelu"), 1.4, 11, "random"),
    S.Workload("diag_big_batch", S.Problem(9000, 128, 128, 48, 2, 500, 1, "bf16", "relu"), 1.1, 11, "none"),
    S.config("C0"),
]


def test_ordinary_build_says_it_has_no_checks():
    assert B.lib().monde_diag_bounds_violations(None, None) == -1


@pytest.mark.parametrize("w", CASES, ids=[w.name for w in CASES])
def test_layers_run_clean_through_the_checking_build(w, monkeypatch):
    p = w.problem
    dev = P.to_device(S.generate(w))
    args = (p, dev["x"], dev["Wg"], dev["bg"], dev["W1"], dev["b1"], dev["W2"], dev["b2"])
    plain = P.run_gpu(p, dev, want_probs=False)
    path = build_mod.build(diagnostics=True)
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", path)
    buf, check = P.guarded_layer_buffers(p)
    out = B.moe_ffn_layer_forward(*args, buf)
    B.monde_poll_device_status(buf.ws)
    check()
    assert _violations()[0] == 0
    assert torch.equal(buf.perm, plain.perm) and torch.equal(out, plain.out)
    if p.dtype == "bf16":
        B.moe_ffn_layer_forward(*args, buf, fuse_combine=True)
        B.monde_poll_device_status(buf.ws)
        check()
        assert _violations()[0] == 0 and torch.equal(buf.out, plain.out)


def test_indices_out_of_range_are_counted_and_skipped(diag_lib):
    w = CASES[0]
    p = w.problem
    dev = P.to_device(S.generate(w))
    buf, check = P.guarded_layer_buffers(p)
    route = lambda: B.monde_route(p, dev["x"], dev["Wg"], dev["bg"], buf.topk_idx, buf.topk_w, buf.counts, buf.offsets,
                                  buf.cls, buf.hot_ids, buf.cold_ids, buf.n_hot_cold, None, buf.ws)
    permute = lambda: B.monde_permute(p, dev["x"], buf.topk_idx, buf.offsets, buf.perm, buf.inv_perm, buf.x_perm, buf.ws)
    A = p.T * p.top_k
    # positions beyond the last row: every assignment of the experts whose offset was moved
    route()
    moved = buf.offsets.clone()
    moved[: p.E] += A
    buf.offsets.copy_(moved)
    permute()
    check()
    n, site, value = _violations()
    assert n == A and site == 2 and value >= A
    # an expert id beyond E in the routing table
    route()
    buf.topk_idx[5, 1] = p.E + 3
    buf.topk_idx[77, 0] = -2
    permute()
    check()
    n, site, value = _violations()
    assert n >= 1 and site == 1 and value in (p.E + 3, -2)
    # a position beyond the last row in the combine
    route()
    permute()
    assert _violations()[0] == 0
    buf.inv_perm[10] = A + 7
    B.monde_combine(p, buf.y_perm.zero_(), buf.inv_perm, buf.topk_w, buf.out)
    check()
    n, site, value = _violations()
    assert n >= 1 and (site, value) == (3, A + 7)        # every thread that handles a piece of that row counts it


def test_an_ffn_unit_out_of_range_is_refused(diag_lib):
    w = CASES[0]
    p = w.problem
    dev = P.to_device(S.generate(w))
    buf, check = P.guarded_layer_buffers(p)
    B.monde_route(p, dev["x"], dev["Wg"], dev["bg"], buf.topk_idx, buf.topk_w, buf.counts, buf.offsets, buf.cls,
                  buf.hot_ids, buf.cold_ids, buf.n_hot_cold, None, buf.ws)
    B.monde_permute(p, dev["x"], buf.topk_idx, buf.offsets, buf.perm, buf.inv_perm, buf.x_perm, buf.ws)
    bad = buf.offsets.clone()
    bad[p.E // 2: p.E] += p.T * p.top_k          # the rows of the upper half of the experts: beyond the buffers
    buf.offsets.copy_(bad)
    L = B.lib()
    L.monde_diag_set_wait_limit_ns(3_000_000)     # units that depend on refused ones give up quickly
    try:
        B.monde_moe_ffn_fwd(p, buf.x_perm, dev["W1"], dev["b1"], dev["W2"], dev["b2"], buf.counts, buf.offsets, buf.cls,
                            buf.hot_ids, buf.cold_ids, buf.n_hot_cold, buf.y_perm, buf.ws)
        with pytest.raises(B.MondeError) as err:
            B.monde_poll_device_status(buf.ws)
    finally:
        L.monde_diag_set_wait_limit_ns(0)
    assert err.value.status in (6, 7)            # out of range (first to be recorded as a rule) or a wait behind it
    check()
    n, site, _ = _violations()
    assert n >= 1 and site == 4
