"""Host-side logic of bench.py: byte and flop counts against the paper's formulas."""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2405_18832_b200 import synthetic as S  # noqa: E402


def test_eq1_reproduces_table2_expert_parameter_sizes():
    # Eq. 1: parameter movement of one MoE layer = 2 * E * d_model * d_ff parameters (bf16: 2 bytes each).
    for line in open(os.path.join(ROOT, "tests", "golden", "table2_expert_params.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, E, d, f, layers, gb = line.split()
        p = S.Problem(1, int(d), int(f), int(E), 1, 1)
        all_active_no_rows = np.ones(int(E), np.int64)
        weights = bench.ffn_algorithmic_bytes(p, all_active_no_rows) - int(E) * (2 * int(d) + 2 * int(f)) * 2
        assert weights == 2 * int(E) * int(d) * int(f) * 2
        assert abs(weights * int(layers) / 1e9 - float(gb)) < 0.06, name


def test_algorithmic_bytes_count_only_activated_experts():
    p = S.Problem(8, 128, 256, 4, 1, 2)
    counts = np.array([5, 0, 3, 0])
    assert bench.ffn_algorithmic_bytes(p, counts) == 2 * 2 * 128 * 256 * 2 + 8 * (2 * 128 + 2 * 256) * 2
    assert bench.ffn_flops(p, counts) == 4 * 8 * 128 * 256


def test_workload_config_names_the_workload():
    cfg = bench.workload_config(S.config("C1"))
    assert "C1" in cfg["workload"] and "model" not in cfg
