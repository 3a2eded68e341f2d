"""CPU checks of bench.py's bookkeeping: the algorithmic byte counts the roofline figures are
built on, the stored DRAM traffic of the dominant kernel against them, and the defaults."""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2605_17862_b200 import synth  # noqa: E402


def test_algorithmic_bytes_of_the_benchmark_workload():
    wl = synth.reasoning()
    aligned = int(wl.mask.sum())
    assert (wl.n_rows, wl.V, aligned) == (32768, 151936, 22040)
    stats, grad = bench.algorithmic_bytes(wl, aligned)
    row = 151936 * 2
    assert stats == 2 * row * aligned == 13_394_677_760
    assert grad == 3 * row * aligned + row * (wl.n_rows - aligned) == 23_351_955_456
    # a gated sample's rows cost a zero fill only
    assert bench.algorithmic_bytes(wl, aligned - 100)[1] == grad - 2 * row * 100


def test_stored_traffic_ratios_and_metric_name():
    # DRAM traffic over algorithmic bytes, from small-case captures: no wasted re-reads
    for name, ratio in bench.NCU_TRAFFIC_RATIO.items():
        assert 0.95 <= ratio <= 1.01, (name, ratio)
    import json
    with open(os.path.join(ROOT, "BASELINE.json")) as fh:
        assert bench.METRIC == json.load(fh)["metric"]


def test_defaults_and_replica_bookkeeping(monkeypatch):
    monkeypatch.setattr(sys, "argv", ["bench.py"])
    args = bench.parse_args()
    assert args.gpus == 1 and args.warmup >= 3 and args.steps >= 20 and args.impl == "fopd"
    assert args.workload == "reasoning" and args.path == "cached"
    value, ms = bench.replica_throughput(22040, 5.0)
    assert ms == 5.0 and abs(value - 22040 / 5e-3) < 1e-6
