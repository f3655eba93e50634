"""The sweep tool: its host-side pieces without a GPU, one tiny run of each sweep with one."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

from paper_2608_19662_b200 import sweep
from paper_2608_19662_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_weight_file_and_pool_index_data():
    w = sweep._load_weights(os.path.join(ROOT, "tests", "golden", "contribution_weights.txt"))
    assert len(w[("Ql", "layer")]) == 36 and len(w[("Qs", "layer")]) == 28
    assert len(w[("Ql", "group")]) == 8 and len(w[("Qs", "group")]) == 8
    assert abs(sum(w[("Ql", "layer")].values()) - 100.0) < 0.5          # printed percentages, rounded to 0.01
    pool = sweep._Pool(wl.QWEN3_4B, 3, 4, 100, True, np.random.default_rng(0))
    assert pool.pool_tokens == 1200 and pool.keep.shape == (1200,) and list(pool.res_off) == [0, 4, 8, 12]
    assert list(pool.slot[:3]) == [0, 100, 200] and all(pool.keep[s + 99] == 1 for s in pool.slot)   # last token kept
    full = sweep._Pool(wl.QWEN3_4B, 1, 2, 50, False, np.random.default_rng(0))
    assert int(full.keep.sum()) == 100


@pytest.mark.gpu
def test_tiny_sweeps_run_and_report_the_printed_sparsities():
    env = dict(os.environ, PYTHONPATH=ROOT)
    out = subprocess.run([sys.executable, "-m", "paper_2608_19662_b200.sweep", "buckets", "--lengths", "512", "--batch", "2",
                          "--tq", "64", "--iters", "2"], capture_output=True, text=True, cwd=ROOT, env=env, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    rec = json.loads(out.stdout.strip().splitlines()[-1])
    assert rec["resource_tokens_per_request"] == 512 and rec["layer_prefill_ms"]["routed_pruned"] > 0
    assert rec["resource_kv_bytes_materialised"]["routed_pruned_zero_copy"] == 0
    assert 0.02 < rec["retained_fraction"] < 0.2
    out = subprocess.run([sys.executable, "-m", "paper_2608_19662_b200.sweep", "budgets", "--budgets", "20,3", "20,7", "--batch", "1",
                          "--n-res", "4", "--res-len", "128", "--tq", "64", "--iters", "1"], capture_output=True, text=True,
                         cwd=ROOT, env=env, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    recs = [json.loads(l) for l in out.stdout.strip().splitlines()]
    rho = {(r["model"], r["k_layers"], r["k_groups"]): r["rho"] for r in recs}
    assert round(100 * rho[("Ql", 20, 3)], 1) == 79.2 and round(100 * rho[("Qs", 20, 7)], 1) == 37.5   # the paper's two budgets
