"""Pins for the CPU oracle: each test ties one part of it to something other than
itself -- a library routine on a special case, a closed form, brute force on tiny
inputs, an invariant, or a hand-worked / tabulated value under tests/golden/."""
import itertools
import math
import os
import random

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    rows = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            parts = line.split()
            rows[parts[0]] = parts[1:]
    return rows


def _rand(rng, *shape, scale=1.0):
    return (rng.standard_normal(shape) * scale).astype(np.float32)


def _to_bf16_bits(a):
    """float32 -> raw bf16 bits (round to nearest even) and the rounded float32."""
    u = a.astype(np.float32).view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    back = (r.astype(np.uint32) << 16).view(np.float32)
    return r, back


# ---------------------------------------------------------------- worked example

def test_hand_worked_example_top1_and_top2():
    g = _golden("worked_example.txt")
    x = np.array([[1, 2]], np.float32)
    Wg = np.eye(2, dtype=np.float32)
    W1 = np.array([[[1, 1], [2, -1]], [[1, -1], [0.5, 0.5]]], np.float32)
    b1 = np.array([[0, 0], [0.5, -1]], np.float32)
    W2 = np.array([[[1, 0], [0, 1]], [[2, 4], [-1, 3]]], np.float32)
    b2 = np.array([[0, 0], [1, 0]], np.float32)
    r1 = oracle.moe_layer(x, Wg, None, W1, b1, W2, b2, 1, 0, 1, "relu")
    assert r1.route.topk_idx.tolist() == [[1]]
    np.testing.assert_allclose(r1.route.probs[0], [float(g["p0"][0]), float(g["p1"][0])], rtol=1e-15)
    np.testing.assert_allclose(r1.out[0], [float(v) for v in g["top1_out"]], rtol=1e-15)
    r2 = oracle.moe_layer(x, Wg, None, W1, b1, W2, b2, 2, 1, 1, "relu")
    assert r2.route.topk_idx.tolist() == [[1, 0]]
    np.testing.assert_allclose(r2.out[0], [float(v) for v in g["top2_out"]], rtol=1e-15)


def test_gelu_is_v_times_normal_cdf():
    # One expert, d = f = 1, W1 = W2 = 1: out = GeLU(x).
    tab = _golden("normal_cdf.txt")
    vs = np.array([[float(v)] for v in tab], np.float32)
    one = np.ones((1, 1, 1), np.float32)
    y = oracle.expert_ffn(vs, np.zeros(len(vs), np.int32), one, None, one, None, "gelu")
    want = np.array([float(v) * float(tab[v][0]) for v in tab])
    np.testing.assert_allclose(y[:, 0], want, rtol=0, atol=2e-16 * 4)
    yr = oracle.expert_ffn(vs, np.zeros(len(vs), np.int32), one, None, one, None, "relu")
    np.testing.assert_array_equal(yr[:, 0], np.maximum(vs[:, 0].astype(np.float64), 0.0))


def test_gelu_approaches_relu_for_large_arguments():
    vs = np.array([[-9.0], [9.0], [-12.5], [12.5]], np.float32)
    one = np.ones((1, 1, 1), np.float32)
    y = oracle.expert_ffn(vs, np.zeros(4, np.int32), one, None, one, None, "gelu")
    np.testing.assert_allclose(y[:, 0], np.maximum(vs[:, 0], 0), atol=1e-15)


# ---------------------------------------------------------------- reductions to a dense FFN

@pytest.mark.parametrize("act", ["relu", "gelu"])
def test_single_expert_is_a_dense_ffn(act):
    rng = np.random.default_rng(1)
    T, d, f = 13, 24, 40
    x, Wg = _rand(rng, T, d), _rand(rng, 1, d)
    W1, b1 = _rand(rng, 1, f, d, scale=0.2), _rand(rng, 1, f, scale=0.3)
    W2, b2 = _rand(rng, 1, d, f, scale=0.2), _rand(rng, 1, d, scale=0.3)
    r = oracle.moe_layer(x, Wg, None, W1, b1, W2, b2, 1, 0, 4, act)
    pre = x.astype(np.float64) @ W1[0].astype(np.float64).T + b1[0]
    if act == "relu":
        h = np.maximum(pre, 0)
    else:
        h = np.array([[0.5 * v * (1 + math.erf(v / math.sqrt(2))) for v in row] for row in pre])
    want = h @ W2[0].astype(np.float64).T + b2[0]
    np.testing.assert_allclose(r.route.topk_w, 1.0, rtol=0, atol=0)
    np.testing.assert_allclose(r.out, want, rtol=1e-12, atol=1e-13)
    assert r.route.counts.tolist() == [T] and r.route.cls.tolist() == [2]


def test_one_hot_gate_bias_sends_every_token_to_one_expert():
    rng = np.random.default_rng(2)
    T, d, f, E, j = 9, 16, 24, 5, 3
    x, Wg = _rand(rng, T, d), _rand(rng, E, d, scale=0.02)
    W1, W2 = _rand(rng, E, f, d, scale=0.2), _rand(rng, E, d, f, scale=0.2)
    b1, b2 = _rand(rng, E, f), _rand(rng, E, d)
    bg = np.zeros(E, np.float32)
    bg[j] = 80.0
    r = oracle.moe_layer(x, Wg, bg, W1, b1, W2, b2, 1, 0, 4, "relu")
    want = np.maximum(x.astype(np.float64) @ W1[j].astype(np.float64).T + b1[j], 0) @ W2[j].astype(np.float64).T + b2[j]
    assert (r.route.topk_idx == j).all()
    np.testing.assert_allclose(r.out, want, rtol=1e-12, atol=1e-13)   # weight = 1 - O(e^-80)
    assert r.route.n_hot_cold.tolist() == [1, 0] and r.route.hot_ids[0] == j


def test_bf16_inputs_are_widened_exactly():
    rng = np.random.default_rng(3)
    T, d, f = 5, 8, 16
    xb, xf = _to_bf16_bits(_rand(rng, T, d))
    W1b, W1f = _to_bf16_bits(_rand(rng, 1, f, d))
    W2b, W2f = _to_bf16_bits(_rand(rng, 1, d, f))
    b1b, b1f = _to_bf16_bits(_rand(rng, 1, f))
    b2b, b2f = _to_bf16_bits(_rand(rng, 1, d))
    e = np.zeros(T, np.int32)
    y16 = oracle.expert_ffn(xb, e, W1b, b1b, W2b, b2b, "relu")
    y32 = oracle.expert_ffn(xf, e, W1f, b1f, W2f, b2f, "relu")
    np.testing.assert_array_equal(y16, y32)
    assert _to_bf16_bits(np.array([1.0, -2.5, 0.33203125], np.float32))[0].tolist() == [0x3F80, 0xC020, 0x3EAA]


# ---------------------------------------------------------------- dense-masked restatement, brute force

def _ffn_py(x, W1, b1, W2, b2, act):
    f, d = len(W1), len(x)
    h = []
    for n in range(f):
        v = b1[n] + sum(x[i] * W1[n][i] for i in range(d))
        h.append(max(v, 0.0) if act == "relu" else 0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0))))
    return [b2[c] + sum(h[n] * W2[c][n] for n in range(f)) for c in range(d)]


def test_dense_masked_restatement_brute_force_on_tiny_problems():
    """out[t] = sum_e G[t,e] * FFN_e(x_t) where G is the sparse gate matrix whose
    support is the k-subset of experts with the largest logit sum (all subsets
    enumerated) and whose values are softmax probabilities (renormalised or not)."""
    py = random.Random(7)
    for trial in range(1000):
        T, E, d, f = py.randint(1, 4), py.randint(1, 4), py.randint(1, 4), py.randint(1, 8)
        k = py.randint(1, min(2, E))
        renorm, act = py.randint(0, 1), py.choice(["relu", "gelu"])
        rng = np.random.default_rng(1000 + trial)
        x, Wg, bg = _rand(rng, T, d), _rand(rng, E, d), _rand(rng, E)
        W1, b1, W2, b2 = _rand(rng, E, f, d), _rand(rng, E, f), _rand(rng, E, d, f), _rand(rng, E, d)
        r = oracle.moe_layer(x, Wg, bg, W1, b1, W2, b2, k, renorm, py.randint(1, 3), act)
        xd, Wgd = x.astype(np.float64).tolist(), Wg.astype(np.float64).tolist()
        for t in range(T):
            l = [float(bg[e]) + sum(xd[t][i] * Wgd[e][i] for i in range(d)) for e in range(E)]
            best = max(itertools.combinations(range(E), k), key=lambda s: sum(l[e] for e in s))
            assert sorted(r.route.topk_idx[t].tolist()) == sorted(best)
            z = sum(math.exp(v - max(l)) for v in l)
            prob = [math.exp(v - max(l)) / z for v in l]
            mass = sum(prob[e] for e in best) if renorm else 1.0
            want = [0.0] * d
            for e in best:
                y = _ffn_py(xd[t], W1[e].astype(np.float64).tolist(), b1[e].astype(np.float64).tolist(),
                            W2[e].astype(np.float64).tolist(), b2[e].astype(np.float64).tolist(), act)
                for c in range(d):
                    want[c] += prob[e] / mass * y[c]
            np.testing.assert_allclose(r.out[t], want, rtol=1e-11, atol=1e-12)


def test_identity_experts_closed_form():
    # W1 = [I;0], W2 = [I 0], no bias, ReLU, x >= 0  =>  FFN_e(x) = x for every e,
    # so out = (sum of gate weights) * x, and exactly x with renormalised top-2.
    rng = np.random.default_rng(5)
    T, d, f, E = 11, 6, 10, 4
    x = np.abs(_rand(rng, T, d))
    Wg = _rand(rng, E, d)
    W1 = np.zeros((E, f, d), np.float32)
    W2 = np.zeros((E, d, f), np.float32)
    for e in range(E):
        W1[e, :d, :] = np.eye(d)
        W2[e, :, :d] = np.eye(d)
    r = oracle.moe_layer(x, Wg, None, W1, None, W2, None, 2, 1, 3, "relu")
    np.testing.assert_allclose(r.out, x.astype(np.float64), rtol=1e-15)
    r = oracle.moe_layer(x, Wg, None, W1, None, W2, None, 2, 0, 3, "relu")
    np.testing.assert_allclose(r.out, x * r.route.topk_w.sum(1, keepdims=True), rtol=1e-15)


# ---------------------------------------------------------------- routing

def test_topk_matches_a_library_sort_and_softmax():
    rng = np.random.default_rng(6)
    T, d, E, k = 200, 12, 17, 4
    x, Wg, bg = _rand(rng, T, d), _rand(rng, E, d), _rand(rng, E)
    r = oracle.route(x, Wg, bg, k, 0, 5)
    l = x.astype(np.float64) @ Wg.astype(np.float64).T + bg
    np.testing.assert_allclose(r.logits, l, rtol=1e-12, atol=1e-13)
    order = np.argsort(-l, axis=1, kind="stable")[:, :k]
    np.testing.assert_array_equal(r.topk_idx, order)
    p = np.exp(l - l.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    np.testing.assert_allclose(r.probs, p, rtol=1e-13)
    np.testing.assert_allclose(r.topk_w, np.take_along_axis(p, order, 1), rtol=1e-13)
    np.testing.assert_allclose(r.probs.sum(1), 1.0, rtol=1e-14)
    # descending slots
    assert (np.diff(np.take_along_axis(l, r.topk_idx, 1), axis=1) <= 0).all()


def test_renormalised_weights_are_a_softmax_over_the_selected_logits():
    rng = np.random.default_rng(8)
    x, Wg = _rand(rng, 50, 9), _rand(rng, 11, 9)
    r = oracle.route(x, Wg, None, 3, 1, 2)
    sel = np.take_along_axis(r.logits, r.topk_idx, 1)
    w = np.exp(sel - sel.max(1, keepdims=True))
    w /= w.sum(1, keepdims=True)
    np.testing.assert_allclose(r.topk_w, w, rtol=1e-13)
    np.testing.assert_allclose(r.topk_w.sum(1), 1.0, rtol=1e-14)
    r1 = oracle.route(x, Wg, None, 1, 1, 2)
    np.testing.assert_array_equal(r1.topk_w, 1.0)
    r0 = oracle.route(x, Wg, None, 1, 0, 2)
    assert (r0.topk_w >= 1.0 / 11).all() and (r0.topk_w <= 1.0).all()


@pytest.mark.parametrize("k,renorm,want", [(1, 0, 1 / 6), (2, 0, 1 / 6), (2, 1, 0.5), (3, 1, 1 / 3)])
def test_uniform_logits_break_ties_toward_small_expert_ids(k, renorm, want):
    x = np.ones((4, 5), np.float32)
    Wg = np.zeros((6, 5), np.float32)
    r = oracle.route(x, Wg, None, k, renorm, 1)
    assert (r.topk_idx == np.arange(k)).all()
    np.testing.assert_allclose(r.topk_w, want, rtol=1e-15)
    assert r.counts.tolist() == [4] * k + [0] * (6 - k)


def test_histogram_scan_classification_and_permutation_invariants():
    rng = np.random.default_rng(9)
    T, d, E, k, theta = 300, 8, 13, 2, 40
    x, Wg = _rand(rng, T, d), _rand(rng, E, d)
    bg = (np.log(np.arange(1, E + 1, dtype=np.float64) ** -1.5) * 1.5).astype(np.float32)
    r = oracle.route(x, Wg, bg, k, 1, theta)
    flat = r.topk_idx.reshape(-1)
    np.testing.assert_array_equal(r.counts, np.bincount(flat, minlength=E))
    assert r.counts.sum() == T * k
    np.testing.assert_array_equal(r.offsets, np.concatenate([[0], np.cumsum(r.counts)]))
    assert (r.topk_idx[:, 0] != r.topk_idx[:, 1]).all()
    cls = np.where(r.counts == 0, 0, np.where(r.counts >= theta, 2, 1))
    np.testing.assert_array_equal(r.cls, cls)
    nh, nc = r.n_hot_cold
    np.testing.assert_array_equal(r.hot_ids[:nh], np.nonzero(cls == 2)[0])
    np.testing.assert_array_equal(r.cold_ids[:nc], np.nonzero(cls == 1)[0])
    assert nh + nc == (r.counts > 0).sum() and nh > 0 and nc > 0
    p = oracle.permute(x, r.topk_idx, r.offsets)
    np.testing.assert_array_equal(p.perm, np.argsort(flat, kind="stable"))
    np.testing.assert_array_equal(np.sort(p.perm), np.arange(T * k))
    np.testing.assert_array_equal(p.inv_perm[p.perm], np.arange(T * k))
    np.testing.assert_array_equal(p.x_perm, x[p.perm // k])
    assert (np.diff(flat[p.perm]) >= 0).all()


@pytest.mark.parametrize("theta,hot,cold", [(0, 3, 0), (1, 3, 0), (2, 2, 1), (5, 1, 2), (6, 0, 3), (1000, 0, 3)])
def test_classification_threshold_edges(theta, hot, cold):
    # counts (5, 1, 0, 2) by construction: expert 2 inactive at every threshold.
    E, d = 4, 4
    Wg = np.eye(E, d, dtype=np.float32) * 10
    who = [0] * 5 + [1] + [3] * 2
    x = np.eye(d, dtype=np.float32)[who]
    r = oracle.route(x, Wg, None, 1, 0, theta)
    assert r.counts.tolist() == [5, 1, 0, 2]
    assert r.n_hot_cold.tolist() == [hot, cold] and r.cls[2] == 0
    assert r.cls[0] == (2 if 5 >= theta else 1)


# ---------------------------------------------------------------- combine

def test_combine_is_a_weighted_gather():
    rng = np.random.default_rng(10)
    T, k, d = 7, 3, 5
    y = rng.standard_normal((T * k, d))
    inv = rng.permutation(T * k).astype(np.int32)
    w = rng.random((T, k))
    out = oracle.combine(y, inv, w)
    want = np.einsum("tk,tkd->td", w, y[inv].reshape(T, k, d))
    np.testing.assert_allclose(out, want, rtol=1e-14)


# ---------------------------------------------------------------- top-H placement (Section 3.3, Eq. 6)

def test_top_h_matches_eq6_worked_by_hand():
    # 10 active of 12 experts; BW_a = 32, BW_b = 96 -> share 32/128 = 1/4.
    counts = np.array([5, 0, 9, 1, 1, 7, 2, 0, 3, 4, 6, 8], np.int32)
    r = oracle.classify_top_h(counts, 1.0, 32.0, 96.0)
    assert r.H == 2                                   # floor(1 * 0.25 * 10) = 2
    assert r.hot_ids[:2].tolist() == [2, 11]          # counts 9 and 8
    assert r.n_hot_cold.tolist() == [2, 8] and r.cls[1] == 0 and r.cls[7] == 0
    assert oracle.classify_top_h(counts, 2.0, 32.0, 96.0).H == 5      # alpha scales H
    assert oracle.classify_top_h(counts, 1.3, 32.0, 96.0).H == 3      # floor(3.25)
    assert oracle.classify_top_h(counts, 0.0, 32.0, 96.0).n_hot_cold.tolist() == [0, 10]
    assert oracle.classify_top_h(counts, 100.0, 32.0, 96.0).n_hot_cold.tolist() == [10, 0]   # clamped to Expert_Activ


def test_top_h_ties_go_to_the_smaller_expert_id_and_balances_the_two_workflows():
    counts = np.array([4, 4, 4, 4, 0, 4, 4], np.int32)
    r = oracle.classify_top_h(counts, 1.0, 1.0, 1.0)          # H = floor(0.5 * 6) = 3
    assert r.hot_ids[:3].tolist() == [0, 1, 2] and r.cold_ids[:3].tolist() == [3, 5, 6]
    # Eq. 4 with equal expert sizes: t_PM ~ H / BW_a, t_MD ~ (Activ - H) / BW_b are balanced by Eq. 6
    active, bw_a, bw_b = 40, 3.0, 5.0
    c = np.arange(1, active + 1, dtype=np.int32)
    H = oracle.classify_top_h(c, 1.0, bw_a, bw_b).H
    assert abs(H / bw_a - (active - H) / bw_b) <= 1.0 / bw_a + 1.0 / bw_b


def test_top_h_equals_the_threshold_rule_at_the_matching_threshold():
    rng = np.random.default_rng(12)
    counts = rng.permutation(np.arange(0, 40)).astype(np.int32)      # distinct counts, one zero
    r = oracle.classify_top_h(counts, 1.0, 1.0, 3.0)                 # H = floor(39 / 4) = 9
    theta = np.sort(counts)[::-1][r.H - 1]
    cls = np.where(counts == 0, 0, np.where(counts >= theta, 2, 1))
    np.testing.assert_array_equal(r.cls, cls)
