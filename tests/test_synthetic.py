"""The seeded input generator: reproducible, device-independent integer core,
near-tie margin honoured, Zipf-shaped histograms like the paper's skew (Section 2.2)."""
import numpy as np
import torch

import oracle
from paper_2405_18832_b200 import synthetic as S


def test_hash_matches_big_integer_reference():
    key = S.stream_key(5, S.TENSOR_W1, 2)
    ctr = torch.tensor([0, 1, 2, 12345678901, (1 << 40) + 7], dtype=torch.int64)
    h = S.hash_u64(key, ctr)
    for c, v in zip(ctr.tolist(), h.tolist()):
        assert (v & S._M64) == S._mix_py(c * S._GOLD + key)


def test_normal_moments_and_chunk_independence():
    key = S.stream_key(0, 0)
    z = S.std_normal(key, torch.arange(1_000_000, dtype=torch.int64))
    assert abs(z.mean().item()) < 5e-3 and abs(z.std().item() - 1) < 5e-3
    a = S.normal_tensor(3, S.TENSOR_W1, (4, 8), 0.02, torch.bfloat16, first=32)
    b = S.normal_tensor(3, S.TENSOR_W1, (2, 4, 8), 0.02, torch.bfloat16)[1]
    assert torch.equal(a, b)


def test_generate_is_deterministic_and_margin_holds():
    for name in ["C0", "C2"]:
        w = S.config(name)
        g1 = S.generate(w, with_weights=(name == "C0"))
        g2 = S.generate(w, with_weights=(name == "C0"))
        for k in g1:
            assert (g1[k] is None and g2[k] is None) or torch.equal(g1[k], g2[k])
        p = w.problem
        r = oracle.route(S.as_numpy(g1["x"]), S.as_numpy(g1["Wg"]), S.as_numpy(g1["bg"]),
                         p.top_k, p.renormalize, p.hot_threshold)
        top = -np.sort(-r.logits, axis=1)[:, : p.top_k + 1]
        assert (top[:, :-1] - top[:, 1:]).min() >= S.NEAR_TIE_MARGIN


def test_zipf_workload_has_a_few_hot_and_many_cold_experts():
    w = S.config("C1")
    g = S.generate(w, with_weights=False)
    p = w.problem
    r = oracle.route(S.as_numpy(g["x"]), S.as_numpy(g["Wg"]), S.as_numpy(g["bg"]), p.top_k, 0, p.hot_threshold)
    nh, nc = r.n_hot_cold
    assert 5 <= nh <= 20 and nc >= 40
    c = np.sort(r.counts)[::-1]
    target = np.arange(1, p.E + 1) ** -1.2
    target = target / target.sum() * p.T
    assert abs(c[0] - target[0]) / target[0] < 0.15


def test_decode_workload_is_all_cold():
    w = S.config("C2")
    g = S.generate(w, with_weights=False)
    p = w.problem
    r = oracle.route(S.as_numpy(g["x"]), S.as_numpy(g["Wg"]), None, 1, 0, p.hot_threshold)
    assert r.n_hot_cold[0] == 0 and 15 <= r.n_hot_cold[1] <= 32 and r.counts.max() <= 6
