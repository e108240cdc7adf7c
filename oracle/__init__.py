"""ctypes front end of the CPU oracle (``monde_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by ``__graft_entry__.smoke()``
and by the CPU-baseline / reference legs of ``bench.py``.  The product path never
touches it.  Arrays are numpy: float32 stays float32, bf16 travels as uint16
holding the raw bits; all results are fp64 / int32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from types import SimpleNamespace
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "monde_oracle.cpp")
_LIB = os.path.join(_HERE, "libmonde_oracle.so")
_lib = None

DT = {"f32": 0, "bf16": 1}
ACT = {"relu": 0, "gelu": 1}


def build(force: bool = False) -> str:
    """Compile the oracle with g++ -O2 (no fast-math, no intrinsics)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_usable_cores.restype = ctypes.c_int
    return _lib


def usable_cores() -> int:
    return int(lib().oracle_usable_cores())


def _p(a: Optional[np.ndarray]):
    if a is None:
        return ctypes.c_void_p(0)
    assert a.flags["C_CONTIGUOUS"]
    return ctypes.c_void_p(a.ctypes.data)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return 0
    if a.dtype == np.uint16:
        return 1
    raise TypeError("oracle inputs are float32 or uint16 (raw bf16 bits), got %s" % a.dtype)


def route(x, Wg, bg, top_k: int, renormalize: int, hot_threshold: int):
    T, d = x.shape
    E = Wg.shape[0]
    dt = _dtype_code(x)
    assert _dtype_code(Wg) == dt and Wg.shape[1] == d
    if bg is not None:
        assert bg.dtype == np.float32 and bg.shape == (E,)
    r = SimpleNamespace(
        logits=np.zeros((T, E), np.float64), probs=np.zeros((T, E), np.float64),
        topk_idx=np.zeros((T, top_k), np.int32), topk_w=np.zeros((T, top_k), np.float64),
        counts=np.zeros(E, np.int32), offsets=np.zeros(E + 1, np.int32), cls=np.zeros(E, np.uint8),
        hot_ids=np.full(E, -1, np.int32), cold_ids=np.full(E, -1, np.int32),
        n_hot_cold=np.zeros(2, np.int32))
    lib().oracle_route(T, d, E, top_k, int(renormalize), int(hot_threshold), dt,
                       _p(x), _p(Wg), _p(bg), _p(r.logits), _p(r.probs), _p(r.topk_idx), _p(r.topk_w),
                       _p(r.counts), _p(r.offsets), _p(r.cls), _p(r.hot_ids), _p(r.cold_ids),
                       _p(r.n_hot_cold))
    return r


def permute(x, topk_idx, offsets):
    T, d = x.shape
    k = topk_idx.shape[1]
    E = offsets.shape[0] - 1
    A = T * k
    perm = np.zeros(A, np.int32)
    inv_perm = np.zeros(A, np.int32)
    x_perm = np.zeros((A, d), x.dtype)
    lib().oracle_permute(T, d, E, k, x.dtype.itemsize, _p(x), _p(np.ascontiguousarray(topk_idx)),
                         _p(offsets), _p(perm), _p(inv_perm), _p(x_perm))
    return SimpleNamespace(perm=perm, inv_perm=inv_perm, x_perm=x_perm)


def expert_ffn(rows, row_expert, W1, b1, W2, b2, act: str, nthreads: int = 0, want_h: bool = False):
    """y[r,:] = FFN_{row_expert[r]}(rows[r,:]) in fp64; optionally also h."""
    n, d = rows.shape
    f = W1.shape[1]
    dt = _dtype_code(rows)
    assert _dtype_code(W1) == dt and _dtype_code(W2) == dt
    assert W1.shape[2] == d and W2.shape[1] == d and W2.shape[2] == f
    row_expert = np.ascontiguousarray(row_expert, np.int32)
    assert row_expert.shape == (n,)
    if n:
        assert row_expert.min() >= 0 and row_expert.max() < W1.shape[0]
    y = np.zeros((n, d), np.float64)
    h = np.zeros((n, f), np.float64) if want_h else None
    lib().oracle_expert_ffn(ctypes.c_int64(n), d, f, ACT[act], dt, _p(rows), _p(row_expert),
                            _p(W1), _p(b1), _p(W2), _p(b2), _p(h), _p(y), int(nthreads))
    return (y, h) if want_h else y


def combine(y_perm, inv_perm, topk_w):
    T, k = topk_w.shape
    d = y_perm.shape[1]
    out = np.zeros((T, d), np.float64)
    lib().oracle_combine(T, d, k, _p(np.ascontiguousarray(y_perm, np.float64)), _p(inv_perm),
                         _p(np.ascontiguousarray(topk_w, np.float64)), _p(out))
    return out


def classify_top_h(counts, alpha: float, bw_a: float, bw_b: float):
    """Hot / cold lists by the paper's top-H rule (Section 3.3, Eq. 6) instead of a threshold."""
    counts = np.ascontiguousarray(counts, np.int32)
    E = counts.shape[0]
    r = SimpleNamespace(cls=np.zeros(E, np.uint8), hot_ids=np.full(E, -1, np.int32),
                        cold_ids=np.full(E, -1, np.int32), n_hot_cold=np.zeros(2, np.int32),
                        H=np.zeros(1, np.int32))
    lib().oracle_classify_top_h(E, _p(counts), ctypes.c_double(alpha), ctypes.c_double(bw_a), ctypes.c_double(bw_b),
                                _p(r.cls), _p(r.hot_ids), _p(r.cold_ids), _p(r.n_hot_cold), _p(r.H))
    r.H = int(r.H[0])
    return r


def experts_of_rows(offsets: np.ndarray) -> np.ndarray:
    """Expert id of every row of the expert-contiguous buffer."""
    return np.repeat(np.arange(offsets.shape[0] - 1, dtype=np.int32), np.diff(offsets)).astype(np.int32)


def moe_layer(x, Wg, bg, W1, b1, W2, b2, top_k: int, renormalize: int, hot_threshold: int,
              act: str, nthreads: int = 0):
    """The whole layer, step by step in the order of Section 2.1."""
    r = route(x, Wg, bg, top_k, renormalize, hot_threshold)
    p = permute(x, r.topk_idx, r.offsets)
    y_perm = expert_ffn(p.x_perm, experts_of_rows(r.offsets), W1, b1, W2, b2, act, nthreads)
    out = combine(y_perm, p.inv_perm, r.topk_w)
    return SimpleNamespace(route=r, perm=p, y_perm=y_perm, out=out)
