"""The parity harness itself, checked on the CPU: a stand-in for the device buffers is filled from the
oracle's own results (rounded to bf16), which the sampled comparison must accept, and then damaged in one
row, which it must reject.  Guards the row / token bookkeeping of the by-expert comparison used for the
layers whose weights exist on the device only."""
from types import SimpleNamespace

import numpy as np
import pytest
import torch

import oracle
import parity as P
from paper_2405_18832_b200 import synthetic as S


def _oracle_buffers(w, g):
    p = w.problem
    h = {k: S.as_numpy(v) for k, v in g.items()}
    ref = oracle.moe_layer(h["x"], h["Wg"], h["bg"], h["W1"], h["b1"], h["W2"], h["b2"], p.top_k, p.renormalize,
                           p.hot_threshold, p.act)
    buf = SimpleNamespace(y_perm=torch.from_numpy(ref.y_perm).to(torch.bfloat16),
                          out=torch.from_numpy(ref.out).to(torch.bfloat16))
    return ref, buf


@pytest.mark.parametrize("sampled", [False, True])
def test_by_expert_comparison_accepts_the_oracle_and_rejects_a_damaged_row(sampled):
    w = S.Workload("harness", S.Problem(400, 128, 256, 12, 2, 16, 1, "bf16", "gelu"), 1.2, 3, "random")
    g = S.generate(w)
    ref, buf = _oracle_buffers(w, g)
    if sampled:
        rows, tokens = P.sample_rows_by_expert(ref.route, ref.perm, w.problem, n_tokens=20, row_budget=200)
        counts = ref.route.counts
        least = np.nonzero(counts > 0)[0][np.argmin(counts[counts > 0])]
        assert set(range(ref.route.offsets[least], ref.route.offsets[least + 1])) <= set(rows.tolist())
        sample = P.OracleSample(w, g, g, ref.route, ref.perm, rows, tokens)
        assert sample.rows.size < w.problem.A and sample.tokens.size == 20
    else:
        sample = P.OracleSample(w, g, g, ref.route, ref.perm)
        assert sample.rows.size == w.problem.A and sample.tokens.size == w.problem.T
    np.testing.assert_allclose(sample.y_ref, ref.y_perm[sample.rows], rtol=0, atol=1e-12)
    np.testing.assert_allclose(sample.out_ref, ref.out[sample.tokens], rtol=0, atol=1e-12)
    sample.compare(buf)
    bad = SimpleNamespace(y_perm=buf.y_perm.clone(), out=buf.out)
    bad.y_perm[int(sample.rows[len(sample.rows) // 2])] *= 1.5
    with pytest.raises(AssertionError):
        sample.compare(bad)
    bad = SimpleNamespace(y_perm=buf.y_perm, out=buf.out.clone())
    bad.out[int(sample.tokens[-1])] += 0.05
    with pytest.raises(AssertionError):
        sample.compare(bad)
