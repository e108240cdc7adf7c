"""GPU parity: the CUDA library (through the C ABI) against the CPU oracle."""
from types import SimpleNamespace

import numpy as np
import pytest
import torch

import oracle
import parity as P
from paper_2405_18832_b200 import binding as B
from paper_2405_18832_b200 import synthetic as S

pytestmark = pytest.mark.gpu


def _wl(name, **kw):
    wl = dict(zipf_alpha=0.0, seed=11, bias="random")
    prob = dict(T=64, d_model=128, d_ff=256, E=8, top_k=1, hot_threshold=8, renormalize=0, dtype="bf16", act="relu")
    for k, v in kw.items():
        (wl if k in wl else prob)[k] = v
    return S.Workload(name, S.Problem(**prob), **wl)


def test_tiny_fp32_config():
    r = P.check_full(S.config("C0"))
    assert r.route.n_hot_cold.sum() == 8


SMALL = [
    _wl("bf16_top1", T=200, d_model=256, d_ff=512, E=16, hot_threshold=16, zipf_alpha=1.2),
    _wl("bf16_top2_renorm_gelu", T=333, d_model=192, d_ff=448, E=12, top_k=2, renormalize=1, act="gelu",
        hot_threshold=40, zipf_alpha=1.0),
    _wl("bf16_ragged_tiles", T=1000, d_model=320, d_ff=832, E=5, top_k=2, hot_threshold=130, zipf_alpha=1.5),
    _wl("bf16_all_hot", T=700, d_model=128, d_ff=256, E=4, top_k=2, hot_threshold=1, renormalize=1),
    _wl("bf16_all_cold", T=40, d_model=256, d_ff=512, E=32, top_k=2, hot_threshold=1000, act="gelu"),
    _wl("bf16_one_token", T=1, d_model=128, d_ff=256, E=8, top_k=2, renormalize=1),
    _wl("bf16_single_expert", T=77, d_model=128, d_ff=192, E=1, top_k=1, hot_threshold=8),
    _wl("bf16_topk_eq_E", T=50, d_model=128, d_ff=128, E=4, top_k=4, renormalize=1, hot_threshold=51),
    _wl("bf16_E256_top8", T=300, d_model=128, d_ff=128, E=256, top_k=8, hot_threshold=12, zipf_alpha=1.0),
    _wl("bf16_no_bias", T=129, d_model=256, d_ff=256, E=8, top_k=1, bias="none", hot_threshold=16),
    _wl("f32_top2_gelu", T=150, d_model=64, d_ff=136, E=6, top_k=2, dtype="f32", act="gelu", renormalize=1,
        hot_threshold=50, zipf_alpha=1.0),
]


@pytest.mark.parametrize("w", SMALL, ids=[w.name for w in SMALL])
def test_small_and_edge_cases_match_the_oracle_elementwise(w):
    P.check_full(w)


@pytest.fixture
def cta_pairs():
    """Runs the expert FFN on CTA pairs (tcgen05 cta_group::2) instead of single CTAs."""
    B.lib().monde_diag_set_ffn_cta_pairs(1)
    yield
    B.lib().monde_diag_set_ffn_cta_pairs(-1)


PAIR_CASES = [w for w in SMALL if w.problem.dtype == "bf16" and w.name in (
    "bf16_top2_renorm_gelu", "bf16_ragged_tiles", "bf16_all_hot", "bf16_all_cold", "bf16_one_token", "bf16_E256_top8")]


@pytest.mark.parametrize("w", PAIR_CASES, ids=[w.name for w in PAIR_CASES])
def test_cta_pair_mode_matches_the_oracle_elementwise(w, cta_pairs):
    # odd feature-tile counts (192 = 1.5 tiles, 832 = 6.5), ragged token tiles, split-K cold tiles
    P.check_full(w)


def test_cta_pair_mode_switch_base_like_layer_full_parity(cta_pairs):
    r = P.check_full(S.config("C1"))
    assert r.out_err[1] < 4e-3


def test_switch_base_like_layer_full_parity():
    r = P.check_full(S.config("C1"))
    assert r.route.n_hot_cold[0] >= 5 and r.route.n_hot_cold[1] >= 40
    assert r.out_err[1] < 4e-3


def test_decode_step_full_parity():
    r = P.check_full(S.config("C2"))
    assert r.route.n_hot_cold[0] == 0


def test_nllb_like_layer_full_parity():
    # every row of y_perm and every token of out against the oracle (2.75e11 flop of fp64 on the host
    # cores: a few tens of seconds), expert weights copied to the host one expert at a time
    w = S.config("C3")
    g = S.generate(w, with_weights=False)
    dev = P.to_device(g)
    dev.update({k: v for k, v in S.generate(w, weights_device="cuda").items() if k in ("W1", "W2", "b1", "b2")})
    r = P.check_by_expert(w, g, dev)
    assert r.full and r.sample.rows.size == 4096 and r.sample.tokens.size == 2048
    assert r.runs[0].route.n_hot_cold[0] >= 15 and r.runs[0].out_err[1] < 4e-3


def test_device_generated_weights_equal_host_generated_ones():
    w = _wl("gen", T=8, d_model=128, d_ff=256, E=3)
    a = S.generate(w)
    b = S.generate(w, weights_device="cuda")
    for k in ("W1", "W2", "b1", "b2"):
        assert torch.equal(a[k], b[k].cpu())


def test_zero_tokens_is_a_no_op():
    p = S.Problem(0, 128, 256, 8, 1, 4)
    buf = B.LayerBuffers(p)
    z = torch.zeros((8, 128), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((8, 256, 128), dtype=torch.bfloat16, device="cuda")
    B.moe_ffn_layer_forward(p, buf.x_dev, z, None, W, None, W.view(8, 128, 256), None, buf)
    B.monde_poll_device_status(buf.ws)
    assert buf.counts.cpu().tolist() == [0] * 8 and buf.n_hot_cold.cpu().tolist() == [0, 0]
    assert buf.offsets.cpu().tolist() == [0] * 9


def test_results_are_bit_reproducible_and_threshold_independent():
    w = _wl("repro", T=500, d_model=256, d_ff=512, E=16, top_k=2, renormalize=1, hot_threshold=30, zipf_alpha=1.2)
    g = S.generate(w)
    dev = P.to_device(g)
    a = P.run_gpu(w.problem, dev)
    b = P.run_gpu(w.problem, dev)
    for name in ("topk_idx", "perm", "inv_perm", "x_perm", "y_perm", "out", "topk_w"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    # the class only selects the kernel: outputs stay within tolerance of each other
    import dataclasses
    for theta in (1, 10 ** 6):
        q = dataclasses.replace(w.problem, hot_threshold=theta)
        c = P.run_gpu(q, dev)
        assert torch.equal(a.perm, c.perm)
        P.check_close("out vs other class", P.widen(c.out), P.widen(a.out), "bf16")


# ---- crossover sweep (E=64, top-2, d_ff = 4 d_model, GELU, renormalised weights) -------------
# Expert outputs do not depend on the threshold, so each (d_model, T, alpha) point is computed once
# by the oracle and every threshold's device output is compared with those oracle values: in full
# where the point is at most 3e11 flop, else on whole experts (one with few rows, one with at least
# 64) plus the rows around a 256-row tile boundary and a token sample.

@pytest.mark.parametrize("d_model", [1024, 2048, 4096])
def test_crossover_sweep_parity_at_every_threshold(d_model):
    weights = None
    for T in (1, 8, 64, 512, 4096):
        for alpha in (0.0, 1.2):
            w = S.sweep_point(d_model, T, alpha, 16)
            g = S.generate(w, with_weights=False)
            dev = P.to_device(g)
            if weights is None:      # same seed and tensor ids at every point of this d_model
                gw = S.generate(w, weights_device="cuda")
                weights = {k: gw[k] for k in ("W1", "W2", "b1", "b2")}
            dev.update(weights)
            r = P.check_by_expert(w, g, dev, thresholds=(4, 16, 64), n_tokens=48, row_budget=384)
            assert r.full == (32.0 * T * d_model * d_model <= 3.0e11)
            assert len(r.runs) == 3 and r.sample.experts_covered.size >= 1


def test_compute_bound_probe_sampled_parity():
    # 8 experts x ~2048 tokens each: every expert hot, many 256-token tiles per expert
    w = S.config("HOTPROBE")
    g = S.generate(w, with_weights=False)
    dev = P.to_device(g)
    dev.update({k: v for k, v in S.generate(w, weights_device="cuda").items() if k in ("W1", "W2", "b1", "b2")})
    r = P.check_sampled(w, g, dev, n_tokens=48)
    assert r.route.n_hot_cold.tolist() == [8, 0]


def test_large_batch_routing_and_permutation_are_bit_exact():
    # 40000 assignments: the two-level recount of the permutation (super-chunks of 2048) is exercised,
    # including a ragged last super-chunk and a ragged last 16-row chunk
    w = _wl("big_batch", T=20000, d_model=128, d_ff=128, E=48, top_k=2, renormalize=1, hot_threshold=500,
            zipf_alpha=1.1, bias="none")
    g = S.generate(w)
    dev = P.to_device(g)
    buf = P.run_gpu(w.problem, dev, want_probs=False)
    P.check_routing(w.problem, g, buf)


def test_host_pipeline_matches_step_by_step_results():
    # five steps with different tokens through the three-stream pipeline (two buffer sets, so every set
    # is reused) must give the bytes that the same steps give one at a time
    w = _wl("pipeline", T=300, d_model=256, d_ff=512, E=16, top_k=2, renormalize=1, hot_threshold=48, zipf_alpha=1.1)
    p = w.problem
    g = S.generate(w)
    dev = P.to_device(g)
    weights = (dev["Wg"], dev["bg"], dev["W1"], dev["b1"], dev["W2"], dev["b2"])
    gen = torch.Generator().manual_seed(5)
    xs = [(g["x"].float() * (1.0 + 0.25 * i) + 0.01 * torch.randn(g["x"].shape, generator=gen)).to(g["x"].dtype).pin_memory()
          for i in range(5)]
    outs = [torch.zeros((p.T, p.d_model), dtype=g["x"].dtype).pin_memory() for _ in xs]
    pipe = B.HostPipeline(p, depth=2)
    for x, o in zip(xs, outs):
        pipe.submit(x, o, *weights)
    pipe.wait()
    buf = B.LayerBuffers(p)
    for x, o in zip(xs, outs):
        ref = B.moe_ffn_layer_forward(p, x.cuda(), *weights, buf)
        torch.cuda.synchronize()
        assert torch.equal(o, ref.cpu())
    assert not torch.equal(outs[0], outs[1])


FUSED_CASES = {
    "C1": lambda: S.config("C1"),
    "C2": lambda: S.config("C2"),
    "ragged_top1": lambda: _wl("ragged_top1", T=777, d_model=320, d_ff=832, E=9, hot_threshold=70, zipf_alpha=1.3, act="gelu"),
    "top2_renorm_gelu": lambda: _wl("top2", T=333, d_model=192, d_ff=448, E=12, top_k=2, renormalize=1, act="gelu",
                                    hot_threshold=40, zipf_alpha=1.0),
    "top4_ragged": lambda: _wl("top4", T=500, d_model=320, d_ff=832, E=10, top_k=4, renormalize=1, hot_threshold=150,
                               zipf_alpha=1.2),
    "C4_d1024_T512": lambda: S.sweep_point(1024, 512, 1.2, 16),
}


@pytest.mark.parametrize("name", list(FUSED_CASES))
def test_fused_combine_gives_the_bytes_of_the_four_call_form(name):
    # top-1: the FFN's last store applies the gate weight and writes `out`; top-k: it stages the rows in token
    # order and the combine kernel adds them without a look-up; either must equal ffn + combine bit for bit
    w = FUSED_CASES[name]()
    p = w.problem
    g = S.generate(w, with_weights=False)
    dev = P.to_device(g)
    dev.update({k: v for k, v in S.generate(w, weights_device="cuda").items() if k in ("W1", "W2", "b1", "b2")})
    weights = (dev["Wg"], dev["bg"], dev["W1"], dev["b1"], dev["W2"], dev["b2"])
    buf = B.LayerBuffers(p)
    ref = B.moe_ffn_layer_forward(p, dev["x"], *weights, buf).clone()
    buf.out.zero_()
    buf.y_perm.fill_(float("nan"))          # the fused form must not depend on y_perm
    got = B.moe_ffn_layer_forward(p, dev["x"], *weights, buf, fuse_combine=True)
    B.monde_poll_device_status(buf.ws)
    assert torch.equal(got, ref)


def test_fused_combine_refuses_fp32():
    w = S.config("C0")
    p = w.problem
    dev = P.to_device(S.generate(w))
    buf = B.LayerBuffers(p)
    with pytest.raises(B.MondeError):
        B.moe_ffn_layer_forward(p, dev["x"], dev["Wg"], dev["bg"], dev["W1"], dev["b1"], dev["W2"], dev["b2"], buf,
                                fuse_combine=True)


def test_one_workspace_serves_alternating_problems():
    # every call leaves the workspace header at zero, so problems of different shapes (different token-tile
    # counts, K-splits, classes) may take turns on one buffer sized for the largest
    wa = _wl("alt_a", T=500, d_model=256, d_ff=1024, E=12, top_k=2, renormalize=1, hot_threshold=40, zipf_alpha=1.2)
    wb = _wl("alt_b", T=90, d_model=384, d_ff=768, E=32, top_k=1, hot_threshold=16, act="gelu")
    runs = []
    for w in (wa, wb):
        g = S.generate(w)
        dev = P.to_device(g)
        fresh = P.run_gpu(w.problem, dev, want_probs=False).out.clone()
        runs.append((w.problem, dev, fresh))
    shared = torch.zeros(max(B.monde_workspace_bytes(p) for p, _, _ in runs), dtype=torch.uint8, device="cuda")
    for p, dev, fresh in runs + runs[::-1] + runs:
        buf = B.LayerBuffers(p)
        buf.ws = shared
        out = B.moe_ffn_layer_forward(p, dev["x"], dev["Wg"], dev["bg"], dev["W1"], dev["b1"], dev["W2"], dev["b2"], buf)
        B.monde_poll_device_status(shared)
        assert torch.equal(out, fresh)
    assert int(shared[:128 * 1024].to(torch.int32).sum()) == 0      # header back at zero


def test_two_layers_on_two_streams_at_once():
    # two persistent launches that cannot both be fully resident: each must still finish (a unit is only
    # ever held by a running CTA) and give the results of running alone
    wa = _wl("conc_a", T=2000, d_model=512, d_ff=2048, E=16, top_k=2, renormalize=1, hot_threshold=64, zipf_alpha=1.2)
    wb = _wl("conc_b", T=1500, d_model=768, d_ff=1536, E=24, top_k=1, hot_threshold=48, zipf_alpha=1.0, act="gelu")
    jobs = []
    for w in (wa, wb):
        dev = P.to_device(S.generate(w))
        alone = P.run_gpu(w.problem, dev, want_probs=False).out.clone()
        jobs.append((w.problem, dev, alone, B.LayerBuffers(w.problem), torch.cuda.Stream()))
    torch.cuda.synchronize()
    for _ in range(10):
        for p, dev, _, buf, st in jobs:
            B.moe_ffn_layer_forward(p, dev["x"], dev["Wg"], dev["bg"], dev["W1"], dev["b1"], dev["W2"], dev["b2"], buf, st)
    for p, dev, alone, buf, st in jobs:
        B.monde_poll_device_status(buf.ws, st)
        assert torch.equal(buf.out, alone)


def test_layer_captured_in_a_cuda_graph_replays_with_new_tokens():
    # decode loops capture the four calls once and replay them: the launches (programmatic dependent launch
    # included) must be capturable and every replay must leave the workspace ready for the next
    w = _wl("graph", T=48, d_model=256, d_ff=1024, E=16, top_k=2, renormalize=1, hot_threshold=12, zipf_alpha=1.0)
    p = w.problem
    g = S.generate(w)
    dev = P.to_device(g)
    weights = (dev["Wg"], dev["bg"], dev["W1"], dev["b1"], dev["W2"], dev["b2"])
    buf = B.LayerBuffers(p)
    x_static = dev["x"].clone()
    B.moe_ffn_layer_forward(p, x_static, *weights, buf)          # first call outside capture (one-time set-up)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            B.moe_ffn_layer_forward(p, x_static, *weights, buf, side)
    eager = B.LayerBuffers(p)
    gen = torch.Generator().manual_seed(9)
    for i in range(4):
        x_new = (g["x"].float() * (1.0 + 0.5 * i) + 0.02 * torch.randn(g["x"].shape, generator=gen)).to(g["x"].dtype).cuda()
        x_static.copy_(x_new)
        graph.replay()
        torch.cuda.synchronize()
        ref = B.moe_ffn_layer_forward(p, x_new, *weights, eager)
        B.monde_poll_device_status(eager.ws)
        assert torch.equal(buf.out, ref)
    B.monde_poll_device_status(buf.ws)


def test_maximum_assignment_count():
    # T * top_k = 2^20, the stated limit: routing, permutation and row gather bit-exact in full (two-level
    # recount over 512 super-chunks), expert outputs on a sample; 16384 assignments per expert on average
    w = _wl("max_A", T=1 << 19, d_model=64, d_ff=128, E=64, top_k=2, renormalize=1, hot_threshold=64,
            zipf_alpha=0.8, bias="none")
    g = S.generate(w)
    dev = P.to_device(g)
    r = P.check_sampled(w, g, dev, n_tokens=256)
    assert int(r.route.counts.sum()) == 1 << 20 and r.route.n_hot_cold[0] == 64


def test_wide_hot_units_with_odd_and_half_feature_tiles():
    # d_model >= 1536 selects two-feature-tile hot units; 1664 = 13 tiles and 1728 = 13.5 tiles leave a last
    # unit with one tile and a tile with 64 valid features, in both layers and both classes
    w = _wl("wide_odd", T=640, d_model=1664, d_ff=1728, E=6, top_k=2, renormalize=1, hot_threshold=100,
            zipf_alpha=1.4, act="gelu")
    r = P.check_full(w)
    assert r.route.n_hot_cold[0] >= 2 and r.route.n_hot_cold[1] >= 1


def test_wide_hot_units_with_odd_and_half_feature_tiles_on_cta_pairs(cta_pairs):
    w = _wl("wide_odd_pairs", T=640, d_model=1664, d_ff=1728, E=6, top_k=2, renormalize=1, hot_threshold=100,
            zipf_alpha=1.4, act="gelu")
    P.check_full(w)


def _ffn_alone(p, counts, seed):
    """monde_moe_ffn_fwd on hand-made per-expert row counts (rows and parameters seeded, drawn here: the
    call needs no router) against the oracle's expert FFN of the same rows."""
    E = p.E
    counts = np.concatenate([np.asarray(counts, np.int64), np.zeros(E - len(counts), np.int64)])   # the rest stay idle
    A = int(counts.sum())
    gen = torch.Generator().manual_seed(seed)
    x_perm = (torch.randn(A, p.d_model, generator=gen) * 1.0).to(torch.bfloat16)
    W1 = (torch.randn(E, p.d_ff, p.d_model, generator=gen) * 0.03).to(torch.bfloat16)
    W2 = (torch.randn(E, p.d_model, p.d_ff, generator=gen) * 0.03).to(torch.bfloat16)
    b1 = (torch.randn(E, p.d_ff, generator=gen) * 0.02).to(torch.bfloat16)
    b2 = (torch.randn(E, p.d_model, generator=gen) * 0.02).to(torch.bfloat16)
    offsets = np.zeros(E + 1, np.int64)
    offsets[1:] = np.cumsum(counts)
    cls = np.where(counts == 0, 0, np.where(counts >= p.hot_threshold, 2, 1)).astype(np.uint8)
    hot = np.flatnonzero(cls == 2)
    cold = np.flatnonzero(cls == 1)
    hot_ids = np.full(E, -1, np.int32)
    cold_ids = np.full(E, -1, np.int32)
    hot_ids[: hot.size] = hot
    cold_ids[: cold.size] = cold
    q = S.Problem(T=A, d_model=p.d_model, d_ff=p.d_ff, E=E, top_k=1, hot_threshold=p.hot_threshold,
                  renormalize=0, dtype="bf16", act=p.act)
    dev = lambda a, dt: torch.as_tensor(a).to(dt).cuda()
    y = torch.full((A, p.d_model), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(B.monde_workspace_bytes(q), dtype=torch.uint8, device="cuda")
    B.monde_moe_ffn_fwd(q, x_perm.cuda(), W1.cuda(), b1.cuda(), W2.cuda(), b2.cuda(), dev(counts, torch.int32),
                        dev(offsets, torch.int32), dev(cls, torch.uint8), dev(hot_ids, torch.int32),
                        dev(cold_ids, torch.int32), dev([hot.size, cold.size], torch.int32), y, ws)
    B.monde_poll_device_status(ws)
    ref = oracle.expert_ffn(S.as_numpy(x_perm), np.repeat(np.arange(E), counts).astype(np.int32), S.as_numpy(W1),
                            S.as_numpy(b1), S.as_numpy(W2), S.as_numpy(b2), p.act)
    got = P.widen(y)
    for e in range(E):          # per expert, so that a small expert's rows are not hidden behind a large one's norm
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        P.check_close(f"expert {e} ({counts[e]} rows)", got[lo:hi], ref[lo:hi], "bf16")


@pytest.mark.parametrize("d_model,d_ff", [(1536, 384), (2048, 320), (512, 384)],
                         ids=["wide_1536", "wide_2048_half_tile", "narrow_512"])
def test_hot_experts_on_either_side_of_the_128_row_sub_class(d_model, d_ff):
    # wide layers (two feature tiles per hot unit) stage hot experts of at most 128 rows through 128-row token
    # tiles after the larger ones; counts sit on both sides of that line and of the 256-row tile, with a large
    # expert whose last tile has fewer than 128 rows (257 = 144 + 113), cold and idle experts in between
    p = S.Problem(T=1, d_model=d_model, d_ff=d_ff, E=14, top_k=1, hot_threshold=32, renormalize=0, dtype="bf16",
                  act="gelu")
    _ffn_alone(p, [128, 129, 0, 257, 31, 32, 300, 1, 127, 256, 0, 513, 33, 16], seed=5)
    _ffn_alone(p, [64, 128, 96], seed=6)            # only the small sub-class
    _ffn_alone(p, [129, 700], seed=7)               # only the large one


@pytest.mark.parametrize("d_model,d_ff", [(1536, 384), (512, 384)], ids=["wide_1536", "narrow_512"])
def test_hot_experts_on_either_side_of_the_128_row_sub_class_on_cta_pairs(d_model, d_ff, cta_pairs):
    p = S.Problem(T=1, d_model=d_model, d_ff=d_ff, E=14, top_k=1, hot_threshold=32, renormalize=0, dtype="bf16",
                  act="relu")
    _ffn_alone(p, [128, 129, 0, 257, 31, 32, 300, 1, 127, 256, 0, 513, 33, 16], seed=8)


def _random_workloads(n, seed, wide_share=0.2, thresholds=(1, 4, 16, 64, 300)):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        big = rng.random() < wide_share
        d_model = int(64 * (rng.integers(24, 37) if big else rng.integers(1, 13)))
        d_ff = int(64 * rng.integers(1, 17 if not big else 9))
        E = int(rng.integers(1, 41))
        top_k = int(rng.integers(1, min(E, 4) + 1))
        out.append(_wl(f"fuzz{i}", T=int(rng.integers(1, 300 if big else 1500)), d_model=d_model, d_ff=d_ff, E=E,
                       top_k=top_k, renormalize=int(rng.integers(0, 2)), hot_threshold=int(rng.choice(list(thresholds))),
                       zipf_alpha=float(rng.choice([0.0, 0.7, 1.2, 1.6])), act=str(rng.choice(["relu", "gelu"])),
                       bias=str(rng.choice(["random", "none"])), seed=100 + i))
    return out


def test_random_shapes_on_one_shared_workspace():
    # 24 seeded random problems (sizes, expert counts, k, thresholds, skew, activation, biases), one after the
    # other on a single workspace, the expert FFN alternately on single CTAs and on CTA pairs, top-1 problems
    # also through the fused-combine entry point; every one against the oracle element by element
    ws = _random_workloads(24, seed=2024)
    shared = torch.zeros(max(B.monde_workspace_bytes(w.problem) for w in ws), dtype=torch.uint8, device="cuda")
    try:
        for i, w in enumerate(ws):
            p = w.problem
            B.lib().monde_diag_set_ffn_cta_pairs(i % 2)
            g = S.generate(w)
            dev = P.to_device(g)
            buf = B.LayerBuffers(p, want_probs=True)
            buf.ws = shared
            B.moe_ffn_layer_forward(p, dev["x"], dev["Wg"], dev["bg"], dev["W1"], dev["b1"], dev["W2"], dev["b2"], buf)
            B.monde_poll_device_status(shared)
            r, pm = P.check_routing(p, g, buf)
            y_ref = oracle.expert_ffn(pm.x_perm, oracle.experts_of_rows(r.offsets), S.as_numpy(g["W1"]), S.as_numpy(g["b1"]),
                                      S.as_numpy(g["W2"]), S.as_numpy(g["b2"]), p.act)
            P.check_close(f"{w.name} y_perm", P.widen(buf.y_perm), y_ref, p.dtype)
            out_ref = oracle.combine(y_ref, pm.inv_perm, r.topk_w)
            P.check_close(f"{w.name} out", P.widen(buf.out), out_ref, p.dtype)
            if p.dtype == "bf16":
                four_calls = buf.out.clone()
                buf.out.zero_()
                B.moe_ffn_layer_forward(p, dev["x"], dev["Wg"], dev["bg"], dev["W1"], dev["b1"], dev["W2"], dev["b2"], buf,
                                        fuse_combine=True)
                B.monde_poll_device_status(shared)
                assert torch.equal(buf.out, four_calls), w.name
    finally:
        B.lib().monde_diag_set_ffn_cta_pairs(-1)


def test_random_wide_shapes_with_hot_experts_of_every_size():
    # 40 seeded random problems, most of them wide (d_model >= 1536: two feature tiles per hot unit, hot experts
    # of at most 128 rows in their own sub-class), thresholds on both sides of 128, single CTAs and CTA pairs in
    # turn; the whole layer against the oracle element by element
    try:
        for i, w in enumerate(_random_workloads(40, seed=4242, wide_share=0.7, thresholds=(1, 4, 16, 33, 64, 129, 300))):
            B.lib().monde_diag_set_ffn_cta_pairs(i % 2)
            P.check_full(w)
    finally:
        B.lib().monde_diag_set_ffn_cta_pairs(-1)


def test_device_status_word_is_reported_and_cleared():
    # the host side of the bounded-wait protocol, with the status word written from the host (no kernel is
    # made to give up): the poll reports it with its site code, clears the whole header, and the workspace
    # serves the next call
    w = S.config("C0")
    p = w.problem
    dev = P.to_device(S.generate(w))
    buf = P.run_gpu(p, dev, want_probs=False)
    good = buf.out.clone()
    hdr = buf.ws[:64].view(torch.int32)
    hdr[0] = 6            # MONDE_ERR_TIMEOUT
    hdr[1] = 5            # a site code
    buf.ws[4096:4100] = 7  # stray counter contents that a half-finished call could leave in the header
    with pytest.raises(B.MondeError) as err:
        B.monde_poll_device_status(buf.ws)
    assert "site 5" in str(err.value) and err.value.status == 6
    assert int(buf.ws[:256 * 1024].to(torch.int32).sum()) == 0
    out = B.moe_ffn_layer_forward(p, dev["x"], dev["Wg"], dev["bg"], dev["W1"], dev["b1"], dev["W2"], dev["b2"], buf)
    B.monde_poll_device_status(buf.ws)
    assert torch.equal(out, good)


# ---- the give-up path of the bounded device waits -------------------------------------------------

@pytest.fixture
def held_rows_and_short_waits():
    """First-layer units never announce their hidden rows and every wait is cut to a few milliseconds,
    so that each second-layer unit's wait for its token tile runs out.  Nothing faults: all accesses
    stay in bounds and the kernel returns by itself."""
    L = B.lib()
    L.monde_diag_set_wait_limit_ns(3_000_000)
    L.monde_diag_set_hold_hidden_ready(1)
    yield
    L.monde_diag_set_hold_hidden_ready(0)
    L.monde_diag_set_wait_limit_ns(0)


def test_a_wait_that_runs_out_is_reported_and_the_workspace_serves_the_next_call(held_rows_and_short_waits):
    w = _wl("give_up", T=500, d_model=256, d_ff=512, E=16, top_k=2, renormalize=1, hot_threshold=30, zipf_alpha=1.2)
    p = w.problem
    dev = P.to_device(S.generate(w))
    args = (p, dev["x"], dev["Wg"], dev["bg"], dev["W1"], dev["b1"], dev["W2"], dev["b2"])
    B.lib().monde_diag_set_hold_hidden_ready(0)
    buf = B.LayerBuffers(p)
    good = B.moe_ffn_layer_forward(*args, buf).clone()
    B.monde_poll_device_status(buf.ws)
    B.lib().monde_diag_set_hold_hidden_ready(1)
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    B.moe_ffn_layer_forward(*args, buf)
    t1.record()
    with pytest.raises(B.MondeError) as err:
        B.monde_poll_device_status(buf.ws)
    assert err.value.status == 6 and "site 5" in str(err.value)      # MONDE_ERR_TIMEOUT, the wait for hidden rows
    assert t0.elapsed_time(t1) < 1000.0                               # the kernel returned by itself, promptly
    assert int(buf.ws[:256 * 1024].to(torch.int32).sum()) == 0        # the poll left the header clean
    B.lib().monde_diag_set_hold_hidden_ready(0)
    again = B.moe_ffn_layer_forward(*args, buf)
    B.monde_poll_device_status(buf.ws)
    assert torch.equal(again, good)


# ---- guard regions around every output (stand-in for a memory checker) ------------------------------

GUARDED = [S.config("C1"), S.config("C2"),
           _wl("ragged_guard", T=1000, d_model=320, d_ff=832, E=5, top_k=2, hot_threshold=130, zipf_alpha=1.5),
           _wl("wide_odd_guard", T=640, d_model=1664, d_ff=1728, E=6, top_k=2, renormalize=1, hot_threshold=100,
               zipf_alpha=1.4, act="gelu"),
           _wl("top1_fused_guard", T=777, d_model=320, d_ff=832, E=9, hot_threshold=70, zipf_alpha=1.3, act="gelu")]


@pytest.mark.parametrize("pairs", [0, 1], ids=["single_ctas", "cta_pairs"])
@pytest.mark.parametrize("w", GUARDED, ids=[w.name for w in GUARDED])
def test_no_kernel_writes_outside_its_outputs(w, pairs):
    p = w.problem
    dev = P.to_device(S.generate(w, with_weights=False))
    dev.update({k: v for k, v in S.generate(w, weights_device="cuda").items() if k in ("W1", "W2", "b1", "b2")})
    args = (p, dev["x"], dev["Wg"], dev["bg"], dev["W1"], dev["b1"], dev["W2"], dev["b2"])
    plain = P.run_gpu(p, dev, want_probs=False)
    B.lib().monde_diag_set_ffn_cta_pairs(pairs)
    try:
        buf, check = P.guarded_layer_buffers(p)
        out = B.moe_ffn_layer_forward(*args, buf)
        B.monde_poll_device_status(buf.ws)
        check()
        assert torch.equal(buf.perm, plain.perm)
        P.check_close("out", P.widen(out), P.widen(plain.out), p.dtype)
        if p.dtype == "bf16":
            B.moe_ffn_layer_forward(*args, buf, fuse_combine=True)
            B.monde_poll_device_status(buf.ws)
            check()
    finally:
        B.lib().monde_diag_set_ffn_cta_pairs(-1)


def test_one_time_setup_is_recorded_per_device():
    L = B.lib()
    w = _wl("setup", T=300, d_model=256, d_ff=512, E=128, top_k=2, renormalize=1, hot_threshold=16, zipf_alpha=1.0)
    inputs = P.to_device(S.generate(w))
    P.run_gpu(w.problem, inputs, want_probs=False)
    dev = torch.cuda.current_device()
    n = L.monde_diag_device_setups(dev)
    assert n >= 1
    P.run_gpu(w.problem, inputs, want_probs=False)
    assert L.monde_diag_device_setups(dev) == n                      # second call: nothing set up again
    assert L.monde_diag_device_setups(dev + 1) == 0                   # a device this process never used
    assert L.monde_diag_device_setups(64) == -1
