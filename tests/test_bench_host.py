"""Host-side pieces of bench.py that need no GPU: the row-parallel run of the CPU oracle must be the oracle's own step."""
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
from oracle import aa_oracle as O  # noqa: E402
from paper_1905_03381_b200 import workloads as W  # noqa: E402


def test_row_parallel_oracle_takes_the_same_steps_as_the_single_threaded_one():
    O.build()
    cfg = W.ImageShape()
    cfg.n, cfg.d = 1500, 96
    x = W.to_oracle(W.uniform01((cfg.n, cfg.d), 100, torch.bfloat16, "cpu"))
    w0 = W.linear_assistant(cfg.d, 2, "cpu")[0].numpy()
    logits = W.normal((cfg.n, cfg.classes), 3.0, 200, torch.float32, "cpu").numpy()
    labels = W.randint(0, cfg.classes, (cfg.n,), 300, "cpu").numpy()
    _, cand1, (w1, b1) = bench.oracle_step_seconds(cfg, x, w0, logits, labels, 3)
    _, cand3, (w3, b3) = bench.oracle_step_seconds_all_cores(cfg, x, w0, logits, labels, 3, 3)
    assert cand1 == cand3 == 3 * cfg.n
    # same batches, same labels; the mean gradient is summed in another order (slices), so fp32 results may differ by an ulp
    assert np.allclose(w1, w3, rtol=1e-6, atol=1e-9) and abs(float(b1) - float(b3)) <= 1e-7
    assert not np.array_equal(w1, w0)


def test_roofline_entries_carry_both_denominators():
    peaks = {"hbm": 6500.0, "burst": 1600.0, "sustained": 1400.0, "kind": "measured"}
    r = bench.hbm_roofline(6.5e9, 2.0, 1.9, 120, peaks, kernel="k")
    assert abs(r["achieved"] - 3250.0) < 1e-9 and abs(r["frac"] - 0.5) < 1e-12 and r["launches_timed"] == 120
    assert abs(r["frac_of_nominal_8TBs"] - 3250.0 / 8000.0) < 1e-12
    t = bench.tensor_roofline(1.6e12, 2.0, 2.0, 50, peaks)
    assert abs(t["achieved"] - 800.0) < 1e-9 and abs(t["frac"] - 0.5) < 1e-12 and abs(t["frac_of_sustained"] - 800 / 1400) < 1e-12
