"""The method sweeps of the benchmark script (fixed draft lengths against Beta-TS, exit depth N,
number of early-exit layers, tree width) run end to end on the tiny configuration: every setting
prints one well-formed line, the quantities are in range and move the way the method says they
must (a fixed draft length is the draft length, a deeper exit accepts at least as much, only trees keep leaves)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _sweep(kind):
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--sweep", kind, "--workload", "tiny-eesd", "--steps", "2"],
                       capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    rows = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    for row in rows:
        assert row["sweep"] == kind and row["workload"] == "tiny-eesd"
        assert row["tokens_per_s"] > 0 and row["speedup_vs_autoregressive"] > 0
        assert 0.0 <= row["v_d"] <= 1.0 and 0.0 <= row["r_d"] <= 1.0 and row["mean_k"] >= 1.0
    return rows


def test_fixed_k_sweep_against_beta_ts():
    rows = _sweep("k")
    assert [r["setting"] for r in rows] == [f"fixed K={K}" for K in range(1, 11)] + ["beta-ts"]
    for K, r in zip(range(1, 11), rows[:10]):
        assert K - 1 < r["mean_k"] <= K                                  # (only the last round of a sequence may be cut short)
    assert 1.0 <= rows[10]["mean_k"] <= 10.0


def test_exit_depth_sweep():
    rows = _sweep("n")
    assert [r["early_layers"] for r in rows] == [1, 2, 3]                # the tiny model has four layers
    assert rows[-1]["v_d"] >= rows[0]["v_d"] - 0.05                      # a deeper exit does not agree less with the target


def test_exit_layer_count_sweep():
    rows = _sweep("exit")
    assert [r["setting"] for r in rows] == ["1 exit layer(s)", "2 exit layer(s)", "3 exit layer(s)"]


def test_tree_width_sweep():
    rows = _sweep("tree")
    assert len(rows) == 3 * 5
    chain = [r for r in rows if r["setting"].startswith("width 1,")]
    wide = [r for r in rows if r["setting"].startswith("width 2,")]
    assert all(r["leaves_kept_per_round"] == 0.0 for r in chain)
    assert any(r["leaves_kept_per_round"] > 0.0 for r in wide)          # the second-best candidate is the target's choice now and then


def test_batch_sweep():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--sweep", "batch", "--workload", "tiny-eesd", "--steps", "1"],
                       capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    rows = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert [(x["sequences"], x["k"]) for x in rows] == [(1, 3), (1, 1), (2, 3), (2, 7), (4, 3), (4, 1), (8, 1)]
    for x in rows:
        assert x["rows_per_verify_pass"] <= 16 and x["tokens_per_s"] > 0 and 0.0 <= x["v_d"] <= 1.0
        assert abs(x["tokens_per_s"] - x["sequences"] * x["tokens_per_s_per_sequence"]) < 0.02 * x["tokens_per_s"]
