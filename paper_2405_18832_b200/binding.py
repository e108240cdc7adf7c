"""Thin ctypes binding of ``libmonde.so``: same names as ``include/monde.h``.

Only argument marshalling happens here (device pointers of torch tensors, the
problem struct, the current CUDA stream).  Every step of the layer runs in the
library's kernels; there is no fallback: if the library is missing or a call
returns a non-zero status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmonde.so")

SYMBOLS = ("monde_workspace_bytes", "monde_status_string", "monde_route", "monde_classify_top_h", "monde_permute",
           "monde_moe_ffn_fwd", "monde_moe_ffn_combine_fwd", "monde_moe_ffn_fwd_static_ws", "monde_combine", "monde_poll_device_status",
           "monde_kernel_launches", "monde_poll_static_ws_status",
           "monde_diag_set_ffn_cta_pairs", "monde_diag_set_trace", "monde_diag_set_wait_limit_ns",
           "monde_diag_set_hold_hidden_ready", "monde_diag_device_setups", "monde_diag_bounds_violations")

_DTYPE = {"f32": 0, "bf16": 1}
_ACT = {"relu": 0, "gelu": 1}


class MondeError(RuntimeError):
    def __init__(self, call: str, status: int):
        self.status = status
        msg = lib().monde_status_string(status).decode()
        super().__init__(f"{call} failed: {msg} (status {status})")


class monde_problem(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("T", "d_model", "d_ff", "E", "top_k", "hot_threshold", "renormalize", "dtype", "act")]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2405_18832_b200.build` (needs nvcc)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32p, f32p = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
        pp = ctypes.POINTER(monde_problem)
        L.monde_workspace_bytes.restype = ctypes.c_size_t
        L.monde_workspace_bytes.argtypes = [pp]
        L.monde_status_string.restype = ctypes.c_char_p
        L.monde_status_string.argtypes = [ctypes.c_int]
        L.monde_route.restype = ctypes.c_int
        L.monde_route.argtypes = [pp, vp, vp, f32p, i32p, f32p, i32p, i32p, vp, i32p, i32p, i32p, f32p,
                                  vp, ctypes.c_size_t, vp]
        L.monde_classify_top_h.restype = ctypes.c_int
        L.monde_classify_top_h.argtypes = [pp, i32p, ctypes.c_double, ctypes.c_double, ctypes.c_double, vp, i32p, i32p,
                                           i32p, vp]
        L.monde_permute.restype = ctypes.c_int
        L.monde_permute.argtypes = [pp, vp, i32p, i32p, i32p, i32p, vp, vp, ctypes.c_size_t, vp]
        L.monde_moe_ffn_fwd.restype = ctypes.c_int
        L.monde_moe_ffn_fwd.argtypes = [pp, vp, vp, vp, vp, vp, i32p, i32p, vp, i32p, i32p, i32p, vp,
                                        vp, ctypes.c_size_t, vp]
        L.monde_moe_ffn_fwd_static_ws.restype = ctypes.c_int
        L.monde_moe_ffn_fwd_static_ws.argtypes = [pp, vp, vp, vp, vp, vp, i32p, i32p, vp, i32p, i32p, i32p, vp, vp]
        L.monde_moe_ffn_combine_fwd.restype = ctypes.c_int
        L.monde_moe_ffn_combine_fwd.argtypes = [pp, vp, vp, vp, vp, vp, i32p, i32p, vp, i32p, f32p, vp, vp,
                                                ctypes.c_size_t, vp]
        L.monde_combine.restype = ctypes.c_int
        L.monde_combine.argtypes = [pp, vp, i32p, f32p, vp, vp]
        L.monde_poll_device_status.restype = ctypes.c_int
        L.monde_poll_device_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32)]
        L.monde_kernel_launches.restype = ctypes.c_longlong
        L.monde_kernel_launches.argtypes = []
        L.monde_poll_static_ws_status.restype = ctypes.c_int
        L.monde_poll_static_ws_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32)]
        L.monde_diag_set_ffn_cta_pairs.restype = None
        L.monde_diag_set_ffn_cta_pairs.argtypes = [ctypes.c_int]
        L.monde_diag_set_trace.restype = None
        L.monde_diag_set_trace.argtypes = [vp, ctypes.c_int]
        L.monde_diag_set_wait_limit_ns.restype = None
        L.monde_diag_set_wait_limit_ns.argtypes = [ctypes.c_ulonglong]
        L.monde_diag_set_hold_hidden_ready.restype = None
        L.monde_diag_set_hold_hidden_ready.argtypes = [ctypes.c_int]
        L.monde_diag_device_setups.restype = ctypes.c_int
        L.monde_diag_device_setups.argtypes = [ctypes.c_int]
        L.monde_diag_bounds_violations.restype = ctypes.c_int
        L.monde_diag_bounds_violations.argtypes = [ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_longlong)]
        _lib = L
    return _lib


def c_problem(p) -> monde_problem:
    """`p`: any object with the fields of monde_problem (dtype / act as names or codes)."""
    dt = p.dtype if isinstance(p.dtype, int) else _DTYPE[p.dtype]
    act = p.act if isinstance(p.act, int) else _ACT[p.act]
    return monde_problem(p.T, p.d_model, p.d_ff, p.E, p.top_k, p.hot_threshold, int(p.renormalize), dt, act)


def _ptr(t: Optional[torch.Tensor]) -> ctypes.c_void_p:
    if t is None:
        return ctypes.c_void_p(0)
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(call: str, status: int) -> None:
    if status != 0:
        raise MondeError(call, status)


def monde_workspace_bytes(p) -> int:
    cp = c_problem(p)
    return int(lib().monde_workspace_bytes(ctypes.byref(cp)))


def monde_route(p, x, Wg, bg, topk_idx, topk_w, counts, offsets, cls, hot_ids, cold_ids, n_hot_cold,
                probs, ws, stream=None) -> None:
    cp = c_problem(p)
    _check("monde_route", lib().monde_route(
        ctypes.byref(cp), _ptr(x), _ptr(Wg), _ptr(bg), _ptr(topk_idx), _ptr(topk_w), _ptr(counts),
        _ptr(offsets), _ptr(cls), _ptr(hot_ids), _ptr(cold_ids), _ptr(n_hot_cold), _ptr(probs),
        _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)))


def monde_classify_top_h(p, counts, alpha, bw_hot_feed, bw_cold_feed, cls, hot_ids, cold_ids, n_hot_cold,
                         stream=None) -> None:
    cp = c_problem(p)
    _check("monde_classify_top_h", lib().monde_classify_top_h(
        ctypes.byref(cp), _ptr(counts), float(alpha), float(bw_hot_feed), float(bw_cold_feed), _ptr(cls),
        _ptr(hot_ids), _ptr(cold_ids), _ptr(n_hot_cold), _stream(stream)))


def monde_permute(p, x, topk_idx, offsets, perm, inv_perm, x_perm, ws, stream=None) -> None:
    cp = c_problem(p)
    _check("monde_permute", lib().monde_permute(
        ctypes.byref(cp), _ptr(x), _ptr(topk_idx), _ptr(offsets), _ptr(perm), _ptr(inv_perm), _ptr(x_perm),
        _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)))


def monde_moe_ffn_fwd(p, x_perm, W1, b1, W2, b2, counts, offsets, cls, hot_ids, cold_ids, n_hot_cold,
                      y_perm, ws, stream=None) -> None:
    cp = c_problem(p)
    _check("monde_moe_ffn_fwd", lib().monde_moe_ffn_fwd(
        ctypes.byref(cp), _ptr(x_perm), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), _ptr(counts), _ptr(offsets),
        _ptr(cls), _ptr(hot_ids), _ptr(cold_ids), _ptr(n_hot_cold), _ptr(y_perm),
        _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)))


def monde_moe_ffn_combine_fwd(p, x_perm, W1, b1, W2, b2, counts, offsets, cls, perm, topk_w, out, ws,
                              stream=None) -> None:
    """Expert FFN and combine in one call, no y_perm (bf16 only): top-1 folds the gate weight into the FFN's
    last store; top-k > 1 stages the rows in token order inside the workspace and adds them in slot order."""
    cp = c_problem(p)
    _check("monde_moe_ffn_combine_fwd", lib().monde_moe_ffn_combine_fwd(
        ctypes.byref(cp), _ptr(x_perm), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), _ptr(counts), _ptr(offsets),
        _ptr(cls), _ptr(perm), _ptr(topk_w), _ptr(out), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)))


STATIC_WS_BYTES = 32 << 20


def monde_moe_ffn_fwd_static_ws(p, x_perm, W1, b1, W2, b2, counts, offsets, cls, hot_ids, cold_ids, n_hot_cold,
                                y_perm, stream=None) -> None:
    """Expert FFN without a caller workspace, for callers that may not allocate device memory
    (pre-allocated serving loops, plug-ins without an allocator): the scratch is a fixed
    array inside the library, shared by all calls on the GPU, so calls must not overlap.
    Raises MondeError(workspace too small) when the problem needs more than STATIC_WS_BYTES."""
    cp = c_problem(p)
    _check("monde_moe_ffn_fwd_static_ws", lib().monde_moe_ffn_fwd_static_ws(
        ctypes.byref(cp), _ptr(x_perm), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), _ptr(counts), _ptr(offsets),
        _ptr(cls), _ptr(hot_ids), _ptr(cold_ids), _ptr(n_hot_cold), _ptr(y_perm), _stream(stream)))


def monde_poll_static_ws_status(stream=None) -> None:
    """monde_poll_device_status for the built-in scratch of monde_moe_ffn_fwd_static_ws: synchronises
    the stream and raises if the last static-workspace call on this GPU recorded a device-side error.
    Ask before the next static-workspace call, which clears the record."""
    site = ctypes.c_int32(0)
    st = lib().monde_poll_static_ws_status(_stream(stream), ctypes.byref(site))
    if st != 0:
        raise MondeError(f"device status of the static workspace (site {site.value})", st)


def monde_combine(p, y_perm, inv_perm, topk_w, out, stream=None) -> None:
    cp = c_problem(p)
    _check("monde_combine", lib().monde_combine(
        ctypes.byref(cp), _ptr(y_perm), _ptr(inv_perm), _ptr(topk_w), _ptr(out), _stream(stream)))


def monde_poll_device_status(ws, stream=None) -> None:
    """Synchronises the stream; raises if a kernel recorded a device-side error."""
    site = ctypes.c_int32(0)
    st = lib().monde_poll_device_status(_ptr(ws), _stream(stream), ctypes.byref(site))
    if st != 0:
        raise MondeError(f"device status (site {site.value})", st)


class LayerBuffers:
    """Device buffers for one layer call, allocated once with torch and reused."""

    def __init__(self, p, device="cuda", want_probs: bool = False):
        dt = torch.bfloat16 if c_problem(p).dtype == 1 else torch.float32
        T, k, E, d = p.T, p.top_k, p.E, p.d_model
        A = T * k
        i32 = dict(dtype=torch.int32, device=device)
        self.topk_idx = torch.empty((T, k), **i32)
        self.topk_w = torch.empty((T, k), dtype=torch.float32, device=device)
        self.counts = torch.empty(E, **i32)
        self.offsets = torch.empty(E + 1, **i32)
        self.cls = torch.empty(E, dtype=torch.uint8, device=device)
        self.hot_ids = torch.full((E,), -1, **i32)
        self.cold_ids = torch.full((E,), -1, **i32)
        self.n_hot_cold = torch.empty(2, **i32)
        self.probs = torch.empty((T, E), dtype=torch.float32, device=device) if want_probs else None
        self.perm = torch.empty(A, **i32)
        self.inv_perm = torch.empty(A, **i32)
        self.x_perm = torch.empty((A, d), dtype=dt, device=device)
        self.y_perm = torch.empty((A, d), dtype=dt, device=device)
        self.out = torch.empty((T, d), dtype=dt, device=device)
        self.ws = torch.zeros(max(monde_workspace_bytes(p), 16), dtype=torch.uint8, device=device)
        self.x_dev = torch.empty((T, d), dtype=dt, device=device)   # staging for host inputs


def moe_ffn_layer_forward(p, x, Wg, bg, W1, b1, W2, b2, buf: LayerBuffers, stream=None,
                          fuse_combine: bool = False) -> torch.Tensor:
    """route -> permute -> expert FFN (hot + cold) -> combine, all enqueued on one stream.
    `fuse_combine` (bf16 problems) takes the three-call form, monde_moe_ffn_combine_fwd: same bytes in `out`,
    no y_perm."""
    monde_route(p, x, Wg, bg, buf.topk_idx, buf.topk_w, buf.counts, buf.offsets, buf.cls, buf.hot_ids,
                buf.cold_ids, buf.n_hot_cold, buf.probs, buf.ws, stream)
    monde_permute(p, x, buf.topk_idx, buf.offsets, buf.perm, buf.inv_perm, buf.x_perm, buf.ws, stream)
    if fuse_combine:
        monde_moe_ffn_combine_fwd(p, buf.x_perm, W1, b1, W2, b2, buf.counts, buf.offsets, buf.cls, buf.perm,
                                  buf.topk_w, buf.out, buf.ws, stream)
        return buf.out
    monde_moe_ffn_fwd(p, buf.x_perm, W1, b1, W2, b2, buf.counts, buf.offsets, buf.cls, buf.hot_ids,
                      buf.cold_ids, buf.n_hot_cold, buf.y_perm, buf.ws, stream)
    monde_combine(p, buf.y_perm, buf.inv_perm, buf.topk_w, buf.out, stream)
    return buf.out


def fused_combine_wins(p) -> bool:
    """Whether monde_moe_ffn_combine_fwd is the faster of the two bit-identical forms of the layer: measured,
    it saves the combine kernel for top-1 routing (2-4 us per layer) and costs time for top-k > 1, where the
    staging rows are written and read like y_perm."""
    cp = c_problem(p)
    return cp.top_k == 1 and cp.dtype == 1


def moe_ffn_layer_forward_host(p, x_host, out_host, Wg, bg, W1, b1, W2, b2, buf: LayerBuffers,
                               stream=None, fuse_combine: bool = False) -> torch.Tensor:
    """Same layer with the step's tokens in pinned host memory: copies them to the device,
    runs the layer, copies the result back and waits for it."""
    buf.x_dev.copy_(x_host, non_blocking=True)
    out = moe_ffn_layer_forward(p, buf.x_dev, Wg, bg, W1, b1, W2, b2, buf, stream, fuse_combine)
    out_host.copy_(out, non_blocking=True)
    (torch.cuda.current_stream() if stream is None else stream).synchronize()
    return out_host


class HostPipeline:
    """Layer steps whose tokens live in pinned host memory, pipelined over three streams.

    The copy of step n+1's tokens to the device and the copy of step n-1's result back to the
    host run while step n computes: `depth` sets of device buffers take turns, events order the
    streams, and the host never waits inside `submit`.  Every step still does its own
    host->device copy, its four calls and its device->host copy; only their overlap across
    steps differs from `moe_ffn_layer_forward_host`.
    """

    def __init__(self, p, depth: int = 2, device="cuda", fuse_combine: bool = False):
        self.p = p
        self.depth = depth
        self.fuse_combine = fuse_combine
        self.bufs = [LayerBuffers(p, device=device) for _ in range(depth)]
        self.s_in = torch.cuda.Stream(device=device)
        self.s_run = torch.cuda.Stream(device=device)
        self.s_out = torch.cuda.Stream(device=device)
        self.copied_in = [torch.cuda.Event() for _ in range(depth)]
        self.computed = [torch.cuda.Event() for _ in range(depth)]
        self.copied_out = [torch.cuda.Event() for _ in range(depth)]
        self.steps = 0

    def submit(self, x_host, out_host, Wg, bg, W1, b1, W2, b2) -> None:
        """Enqueues one step; `out_host` holds its result once `wait()` (or a later event) says so."""
        i = self.steps % self.depth
        buf = self.bufs[i]
        reused = self.steps >= self.depth
        if reused:
            self.s_in.wait_event(self.computed[i])        # the step that last read this x_dev has run
        with torch.cuda.stream(self.s_in):
            buf.x_dev.copy_(x_host, non_blocking=True)
        self.copied_in[i].record(self.s_in)
        self.s_run.wait_event(self.copied_in[i])
        if reused:
            self.s_run.wait_event(self.copied_out[i])     # this buffer set's previous result has left
        moe_ffn_layer_forward(self.p, buf.x_dev, Wg, bg, W1, b1, W2, b2, buf, self.s_run, self.fuse_combine)
        self.computed[i].record(self.s_run)
        self.s_out.wait_event(self.computed[i])
        with torch.cuda.stream(self.s_out):
            out_host.copy_(buf.out, non_blocking=True)
        self.copied_out[i].record(self.s_out)
        self.steps += 1

    def wait(self) -> None:
        self.s_out.synchronize()
        for buf in self.bufs:
            monde_poll_device_status(buf.ws, self.s_run)
