"""Seeded synthetic inputs for the MoE FFN layer (tokens, gate, expert weights).

This module is the one piece shared by the CPU oracle's tests and the CUDA
path's tests: it only *draws inputs*.  It holds none of the layer's arithmetic
that is under test; the one matrix product it forms (gate logits, through a
library matmul in fp64) is used solely to shape the inputs -- to calibrate the
gate bias toward a Zipf expert popularity and to re-draw tokens whose top
logits are nearly tied -- and its result is never handed to either side.

The inputs stand in for the paper's workloads (Table 2: Switch-Large-128 with
top-1 gating, NLLB-MoE with top-2 gating, bf16, skewed token-to-expert
distribution as in Section 2.2 / Fig. 3).  The trained weights and the XSum /
FLORES-200 data are not available, so shapes and skew follow the paper while
values are random.

Every value is a pure function of (seed, tensor id, draw, element index): a
counter-based generator written with exact integer operations followed by one
correctly rounded multiply, so the CPU and a CUDA device produce bit-identical
tensors.  That lets multi-gigabyte expert weights be drawn directly in device
memory while the oracle reads the very same bytes.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import numpy as np
import torch

_M64 = (1 << 64) - 1
_GOLD = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB
_K_SEED = 0xD6E8FEB86659FD93
_K_TENSOR = 0xA0761D6478BD642F
_K_DRAW = 0xE7037ED1A0B428DB
_K_SECOND = 0x8EBC6AF09C88C6E3

NEAR_TIE_MARGIN = 1e-2  # minimum gap between adjacent logits among ranks 1..k+1

TENSOR_X, TENSOR_WG, TENSOR_W1, TENSOR_W2, TENSOR_B1, TENSOR_B2, TENSOR_ORDER = range(7)


def _s64(v: int) -> int:
    """Python int -> the same 64 bits read as a signed value (for torch.int64)."""
    v &= _M64
    return v - (1 << 64) if v >= (1 << 63) else v


def _mix_py(z: int) -> int:
    """splitmix64 finaliser on Python ints (reference for the tensor version)."""
    z &= _M64
    z = ((z ^ (z >> 30)) * _C1) & _M64
    z = ((z ^ (z >> 27)) * _C2) & _M64
    return z ^ (z >> 31)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _s64(_C1)
    z = (z ^ _lsr(z, 27)) * _s64(_C2)
    return z ^ _lsr(z, 31)


def stream_key(seed: int, tensor_id: int, draw: int = 0) -> int:
    return _mix_py(seed * _K_SEED + tensor_id * _K_TENSOR + draw * _K_DRAW + 1)


def hash_u64(key: int, ctr: torch.Tensor) -> torch.Tensor:
    """64 hashed bits per counter value (int64 tensor holding the raw bits)."""
    return _mix(ctr * _s64(_GOLD) + _s64(key))


_SUM_MEAN = 4 * 65535  # mean of a sum of eight uniform draws on 0..65535
_SUM_STD = math.sqrt(8.0 * (65536.0 ** 2 - 1.0) / 12.0)


def std_normal(key: int, ctr: torch.Tensor) -> torch.Tensor:
    """Approximately N(0,1) values in float64, one per counter.

    Sum of eight 16-bit uniform fields taken from two hashed words, centred and
    scaled to unit variance (Irwin-Hall with n=8: excess kurtosis -0.15, support
    +-4.9 sigma).  Integer arithmetic is exact, so every device agrees bit for bit.
    """
    h1 = hash_u64(key, ctr)
    h2 = _mix(h1 + _s64(_K_SECOND))
    s = torch.zeros_like(ctr)
    for h in (h1, h2):
        for sh in (0, 16, 32, 48):
            s = s + ((h >> sh) & 0xFFFF)
    return (s - _SUM_MEAN).to(torch.float64) * (1.0 / _SUM_STD)


def normal_tensor(seed: int, tensor_id: int, shape, std: float, dtype: torch.dtype,
                  device="cpu", draw: int = 0, first: int = 0) -> torch.Tensor:
    """std * N(0,1) for flat element indices first .. first+numel-1, rounded once
    to float32 and once more to `dtype`."""
    n = int(np.prod(shape))
    ctr = torch.arange(first, first + n, dtype=torch.int64, device=device)
    z = std_normal(stream_key(seed, tensor_id, draw), ctr)
    return (z * std).to(torch.float32).to(dtype).reshape(shape)


# ----------------------------------------------------------------------------
# Problem / workload descriptions
# ----------------------------------------------------------------------------

@dataclasses.dataclass(frozen=True)
class Problem:
    """Layer dimensions in the paper's notation (Table 1); T = B*S tokens."""
    T: int
    d_model: int
    d_ff: int
    E: int
    top_k: int
    hot_threshold: int
    renormalize: int = 0
    dtype: str = "bf16"      # "bf16" or "f32"
    act: str = "relu"        # "relu" or "gelu"

    @property
    def A(self) -> int:
        return self.T * self.top_k

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 4


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    problem: Problem
    zipf_alpha: float = 0.0   # 0 -> no gate bias (uniform popularity)
    seed: int = 0
    bias: str = "none"        # "none" (null pointers) | "zero" | "random"
    bias_std: float = 0.02


def config(name: str) -> Workload:
    """The named workloads (shapes of the paper's Table 2 models, synthetic values)."""
    if name == "C0":   # tiny fp32 parity case
        return Workload("C0", Problem(64, 128, 512, 8, 1, 8, 0, "f32", "relu"), 0.0, 0, "zero")
    if name == "C1":   # Switch-Base-like encoder layer
        return Workload("C1", Problem(4096, 768, 3072, 64, 1, 64, 0, "bf16", "relu"), 1.2, 1)
    if name == "C2":   # Switch-Large-like decode step
        return Workload("C2", Problem(32, 1024, 4096, 128, 1, 16, 0, "bf16", "relu"), 0.0, 2)
    if name == "C3":   # NLLB-MoE-like layer
        return Workload("C3", Problem(2048, 2048, 8192, 128, 2, 32, 1, "bf16", "relu"), 1.0, 3)
    if name == "HOTPROBE":   # compute-bound probe of the hot tiling: 8 experts x ~2048 tokens, NLLB-sized FFN
        return Workload("HOTPROBE", Problem(16384, 2048, 8192, 8, 1, 32, 0, "bf16", "relu"), 0.0, 5)
    raise KeyError(name)


def sweep_point(d_model: int, T: int, alpha: float, theta: int, seed: int = 4) -> Workload:
    """One point of the hot/cold crossover sweep (E=64, top-2, d_ff=4*d_model, GELU)."""
    p = Problem(T, d_model, 4 * d_model, 64, 2, theta, 1, "bf16", "gelu")
    return Workload(f"C4_d{d_model}_T{T}_a{alpha}_th{theta}", p, alpha, seed)


# ----------------------------------------------------------------------------
# Generation
# ----------------------------------------------------------------------------

def _logits64(x: torch.Tensor, Wg: torch.Tensor, bg: Optional[torch.Tensor]) -> torch.Tensor:
    l = x.to(torch.float64) @ Wg.to(torch.float64).T
    if bg is not None:
        l = l + bg.to(torch.float64)
    return l


def zipf_target(E: int, alpha: float, seed: int) -> torch.Tensor:
    """Target popularity p_e: rank r gets r^-alpha, ranks dealt to expert ids by a
    seeded shuffle so that popular experts are not contiguous."""
    key = stream_key(seed, TENSOR_ORDER)
    h = hash_u64(key, torch.arange(E, dtype=torch.int64))
    order = torch.argsort(h, stable=True)          # order[r] = expert holding rank r+1
    p_rank = torch.arange(1, E + 1, dtype=torch.float64) ** (-alpha)
    p_rank = p_rank / p_rank.sum()
    p = torch.empty(E, dtype=torch.float64)
    p[order] = p_rank
    return p


def _has_near_tie(l: torch.Tensor, k: int) -> torch.Tensor:
    E = l.shape[1]
    top = torch.sort(l, dim=1, descending=True).values[:, : min(k + 1, E)]
    if top.shape[1] < 2:
        return torch.zeros(l.shape[0], dtype=torch.bool)
    gaps = top[:, :-1] - top[:, 1:]
    return (gaps < NEAR_TIE_MARGIN).any(dim=1)


def generate(w: Workload, weights_device="cpu", with_weights: bool = True) -> Dict[str, Optional[torch.Tensor]]:
    """Draw all layer inputs.  x, Wg, bg live on the CPU; expert weights are drawn on
    `weights_device` (same bits on any device)."""
    p = w.problem
    dt = p.torch_dtype
    T, d, f, E, k = p.T, p.d_model, p.d_ff, p.E, p.top_k
    Wg = normal_tensor(w.seed, TENSOR_WG, (E, d), 0.02, dt)
    x = normal_tensor(w.seed, TENSOR_X, (T, d), 1.0, dt)

    bg = None
    if w.zipf_alpha > 0.0 and E > 1:
        target = zipf_target(E, w.zipf_alpha, w.seed)
        beta = 0.02 * math.sqrt(d) * math.sqrt(6.0) / math.pi
        bg = (beta * torch.log(target)).to(torch.float32)
        for _ in range(8):   # pull the empirical top-1 frequency toward the target
            top1 = torch.argmax(_logits64(x, Wg, bg), dim=1)
            freq = torch.bincount(top1, minlength=E).to(torch.float64) / T
            freq = torch.clamp(freq, min=0.5 / T)
            bg = (bg.to(torch.float64) + 0.5 * beta * (torch.log(target) - torch.log(freq))).to(torch.float32)

    # Re-draw tokens whose top logits are nearly tied, so that fp32 accumulation
    # order can never change the routing decision.
    for draw in range(1, 200):
        bad = _has_near_tie(_logits64(x, Wg, bg), k)
        idx = torch.nonzero(bad).flatten()
        if idx.numel() == 0:
            break
        ctr = (idx[:, None] * d + torch.arange(d, dtype=torch.int64)[None, :]).reshape(-1)
        z = std_normal(stream_key(w.seed, TENSOR_X, draw), ctr)
        x[idx] = z.to(torch.float32).to(dt).reshape(-1, d)
    else:
        raise RuntimeError("near-tie rejection did not converge")

    out: Dict[str, Optional[torch.Tensor]] = {"x": x, "Wg": Wg, "bg": bg,
                                              "W1": None, "b1": None, "W2": None, "b2": None}
    if with_weights:
        W1 = torch.empty((E, f, d), dtype=dt, device=weights_device)
        W2 = torch.empty((E, d, f), dtype=dt, device=weights_device)
        for e in range(E):
            W1[e] = normal_tensor(w.seed, TENSOR_W1, (f, d), 0.02, dt, weights_device, first=e * f * d)
            W2[e] = normal_tensor(w.seed, TENSOR_W2, (d, f), 0.02, dt, weights_device, first=e * f * d)
        out["W1"], out["W2"] = W1, W2
        if w.bias == "zero":
            out["b1"] = torch.zeros((E, f), dtype=dt, device=weights_device)
            out["b2"] = torch.zeros((E, d), dtype=dt, device=weights_device)
        elif w.bias == "random":
            out["b1"] = normal_tensor(w.seed, TENSOR_B1, (E, f), w.bias_std, dt, weights_device)
            out["b2"] = normal_tensor(w.seed, TENSOR_B2, (E, d), w.bias_std, dt, weights_device)
    return out


def as_numpy(t: Optional[torch.Tensor]) -> Optional[np.ndarray]:
    """Host view of a tensor's bytes: float32 stays float32, bf16 becomes uint16."""
    if t is None:
        return None
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
