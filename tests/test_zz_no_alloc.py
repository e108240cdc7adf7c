"""The allocation-free expert FFN entry point (scratch in a fixed array inside the library).

It serves callers that cannot call cudaMalloc where the layer runs - a serving loop that
pre-allocates everything, a plug-in that is handed its buffers - so the test calls it through
the C ABI with caller-owned inputs and outputs only, twice in a row (the second call finds the
first call's leftovers in the shared array), and compares with the ordinary entry point.
This file is collected last on purpose: a failure here cannot hide any other test's result.
"""
import ctypes

import numpy as np
import pytest
import torch

import parity as P
from paper_2405_18832_b200 import binding as B
from paper_2405_18832_b200 import synthetic as S


def _route_and_permute(p, dev):
    buf = B.LayerBuffers(p)
    B.monde_route(p, dev["x"], dev["Wg"], dev["bg"], buf.topk_idx, buf.topk_w, buf.counts, buf.offsets, buf.cls,
                  buf.hot_ids, buf.cold_ids, buf.n_hot_cold, None, buf.ws)
    B.monde_permute(p, dev["x"], buf.topk_idx, buf.offsets, buf.perm, buf.inv_perm, buf.x_perm, buf.ws)
    return buf


CASES = [
    S.config("C2"),                                                      # decode step, all cold, split-K
    S.Workload("mixed", S.Problem(300, 256, 1024, 16, 2, 24, 1, "bf16", "gelu"), 1.2, 21, "random"),
    S.config("C0"),                                                      # fp32 path
]


@pytest.mark.gpu
@pytest.mark.parametrize("w", CASES, ids=[w.name for w in CASES])
def test_static_workspace_entry_point_matches_the_ordinary_one_twice(w):
    p = w.problem
    assert B.monde_workspace_bytes(p) <= B.STATIC_WS_BYTES
    g = S.generate(w, with_weights=False)
    gw = S.generate(w, weights_device="cuda")
    dev = P.to_device(g)
    dev.update({k: gw[k] for k in ("W1", "W2", "b1", "b2")})
    buf = _route_and_permute(p, dev)
    args = (p, buf.x_perm, dev["W1"], dev["b1"], dev["W2"], dev["b2"], buf.counts, buf.offsets, buf.cls,
            buf.hot_ids, buf.cold_ids, buf.n_hot_cold)
    B.monde_moe_ffn_fwd(*args, buf.y_perm, buf.ws)
    B.monde_poll_device_status(buf.ws)
    want = buf.y_perm.clone()
    for call in range(2):
        y = torch.full_like(buf.y_perm, float("nan"))
        B.monde_moe_ffn_fwd_static_ws(*args, y)
        B.monde_poll_static_ws_status()          # synchronises; raises if a device-side wait gave up
        assert torch.equal(y, want), f"static-ws call {call}"      # same kernels, same order of sums: same bytes


@pytest.mark.gpu
def test_a_timeout_inside_a_static_workspace_call_reaches_the_caller():
    # the caller cannot see the built-in array, so a wait that ran out is reported by the array's own poll;
    # made to happen by the diagnostic switches (rows never announced, waits cut to 3 ms), nothing faults
    w = CASES[1]
    p = w.problem
    g = S.generate(w, with_weights=False)
    dev = P.to_device(g)
    dev.update({k: v for k, v in S.generate(w, weights_device="cuda").items() if k in ("W1", "W2", "b1", "b2")})
    buf = _route_and_permute(p, dev)
    args = (p, buf.x_perm, dev["W1"], dev["b1"], dev["W2"], dev["b2"], buf.counts, buf.offsets, buf.cls,
            buf.hot_ids, buf.cold_ids, buf.n_hot_cold)
    y = torch.empty_like(buf.y_perm)
    B.monde_moe_ffn_fwd_static_ws(*args, y)
    B.monde_poll_static_ws_status()
    good = y.clone()
    L = B.lib()
    L.monde_diag_set_wait_limit_ns(3_000_000)
    L.monde_diag_set_hold_hidden_ready(1)
    try:
        B.monde_moe_ffn_fwd_static_ws(*args, y)
        with pytest.raises(B.MondeError) as err:
            B.monde_poll_static_ws_status()
        assert err.value.status == 6 and "site 5" in str(err.value)
    finally:
        L.monde_diag_set_hold_hidden_ready(0)
        L.monde_diag_set_wait_limit_ns(0)
    B.monde_poll_static_ws_status()              # the report cleared the record
    B.monde_moe_ffn_fwd_static_ws(*args, y)
    B.monde_poll_static_ws_status()
    assert torch.equal(y, good)


@pytest.mark.gpu
def test_static_workspace_entry_point_rejects_problems_beyond_its_limit():
    p = S.config("C1").problem
    assert B.monde_workspace_bytes(p) > B.STATIC_WS_BYTES
    cp = B.c_problem(p)
    a = ctypes.c_void_p(4096)   # never dereferenced: the size check comes first
    st = B.lib().monde_moe_ffn_fwd_static_ws(ctypes.byref(cp), a, a, a, a, a, a, a, a, a, a, a, a, None)
    assert st == 3 and b"workspace" in B.lib().monde_status_string(st)
