"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
symbol the public header declares, sizes its workspace, and rejects bad arguments
before any launch."""
import ctypes
import os
import re
from types import SimpleNamespace

import pytest

from paper_2405_18832_b200 import binding as B
from paper_2405_18832_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build_mod.build()
    return B.lib()


def _declared_functions():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(monde_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol(L):
    declared = _declared_functions()
    assert set(B.SYMBOLS) <= set(declared) and len(declared) >= 7
    for name in declared:
        assert hasattr(L, name), name


def _problem(**kw):
    base = dict(T=64, d_model=128, d_ff=512, E=8, top_k=1, hot_threshold=8, renormalize=0, dtype="bf16", act="relu")
    base.update(kw)
    return SimpleNamespace(**base)


def test_workspace_bytes_covers_the_hidden_activations(L):
    p = _problem()
    n = B.monde_workspace_bytes(p)
    assert n >= p.T * p.top_k * p.d_ff * 2
    assert B.monde_workspace_bytes(_problem(dtype="f32")) >= p.T * p.d_ff * 4
    assert B.monde_workspace_bytes(_problem(T=0)) > 0


@pytest.mark.parametrize("bad", [dict(top_k=9, E=8), dict(top_k=0), dict(E=0), dict(d_model=0), dict(T=-1),
                                 dict(E=257, top_k=1), dict(d_model=96), dict(d_ff=100), dict(dtype=7), dict(act=5),
                                 dict(top_k=9, E=64)])
def test_invalid_problems_are_rejected_on_the_host(L, bad):
    p = _problem(**bad)
    assert B.monde_workspace_bytes(p) == 0
    cp = B.c_problem(p)
    z = ctypes.c_void_p(0)
    st = L.monde_combine(ctypes.byref(cp), z, z, z, z, z)
    assert st in (1, 2)


def test_null_pointers_are_rejected_before_any_launch(L):
    cp = B.c_problem(_problem())
    z = ctypes.c_void_p(0)
    assert L.monde_combine(ctypes.byref(cp), z, z, z, z, z) == 1
    assert L.monde_permute(ctypes.byref(cp), z, z, z, z, z, z, z, 0, z) == 1
    assert L.monde_moe_ffn_fwd(ctypes.byref(cp), z, z, z, z, z, z, z, z, z, z, z, z, z, 0, z) == 1
    assert L.monde_route(ctypes.byref(cp), z, z, z, z, z, z, z, z, z, z, z, z, z, 0, z) == 1
    assert L.monde_poll_device_status(z, z, None) == 1
    assert L.monde_route(None, z, z, z, z, z, z, z, z, z, z, z, z, z, 0, z) == 1


def test_misaligned_pointer_and_small_workspace(L):
    cp = B.c_problem(_problem())
    a = ctypes.c_void_p(4096)      # never dereferenced: checks run first
    odd = ctypes.c_void_p(4100)
    z = ctypes.c_void_p(0)
    assert L.monde_combine(ctypes.byref(cp), odd, a, a, a, z) == 1
    assert L.monde_permute(ctypes.byref(cp), a, a, a, a, a, a, a, 16, z) == 3


def test_fused_combine_entry_point_checks_its_arguments_on_the_host(L):
    z = ctypes.c_void_p(0)
    a = ctypes.c_void_p(4096)      # never dereferenced: checks run first
    args = lambda cp: (ctypes.byref(cp), a, a, z, a, z, a, a, a, a, a, a, a, 1 << 30, z)
    assert L.monde_moe_ffn_combine_fwd(*args(B.c_problem(_problem(dtype="f32")))) == 2   # bf16 only
    cp = B.c_problem(_problem())
    assert L.monde_moe_ffn_combine_fwd(ctypes.byref(cp), a, a, z, a, z, a, a, a, z, a, a, a, 1 << 30, z) == 1   # perm missing
    assert L.monde_moe_ffn_combine_fwd(ctypes.byref(cp), a, a, z, a, z, a, a, a, a, a, a, a, 16, z) == 3       # workspace too small


def test_diagnostic_switches_and_per_device_bookkeeping(L):
    # nothing has been launched in this process: no device has had its one-time set-up
    assert [L.monde_diag_device_setups(d) for d in (0, 1, 63)] == [0, 0, 0]
    assert L.monde_diag_device_setups(-1) == -1 and L.monde_diag_device_setups(64) == -1
    # the switches only record values; defaults come back with the documented arguments
    L.monde_diag_set_wait_limit_ns(5_000_000)
    L.monde_diag_set_wait_limit_ns(0)
    L.monde_diag_set_hold_hidden_ready(1)
    L.monde_diag_set_hold_hidden_ready(0)
    L.monde_diag_set_ffn_cta_pairs(1)
    L.monde_diag_set_ffn_cta_pairs(-1)
    L.monde_diag_set_trace(None, 0)


def test_static_workspace_poll_needs_a_device(L):
    # without a CUDA device the array's address cannot be looked up: a CUDA error status, not a crash
    import torch
    if not torch.cuda.is_available():
        assert L.monde_poll_static_ws_status(None, None) == 5


def test_status_strings(L):
    assert L.monde_status_string(0) == b"ok"
    assert b"timed out" in L.monde_status_string(6)
    assert L.monde_status_string(99) == b"unknown status"


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libmonde.so"))
    with pytest.raises(RuntimeError, match="missing"):
        B.lib()
