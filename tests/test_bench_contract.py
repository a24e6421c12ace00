"""The benchmark's output contract: one JSON line with the agreed keys, for the reference arm (CPU, runs anywhere)
and for the GPU arm (short run)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config"}


def _run(args, timeout):
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                       timeout=timeout, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1, p.stdout[-2000:]
    return json.loads(lines[0])


def test_reference_arm_prints_the_contract_line():
    d = _run(["--impl", "reference", "--steps", "1", "--warmup", "1"], timeout=300)
    assert BASE_KEYS <= set(d) and d["impl"] == "reference" and d["higher_is_better"] is True
    assert d["metric"] == "kv_token_heads_attended_per_s" and d["unit"] == "token-heads/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and "sample" in d["cpu_baseline"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["vs_baseline"] is None and "workload" in d["config"]
    sys.path.insert(0, ROOT)
    import bench
    assert set(d["config"]) == set(bench.CONFIG_KEYS)    # the same keys as the GPU arm prints (None where not applicable)


@pytest.mark.gpu
def test_gpu_arm_prints_the_contract_line():
    d = _run(["--steps", "8", "--warmup", "3", "--prep-rounds", "1", "--no-cpu-baseline", "--no-per-layer"], timeout=900)
    assert BASE_KEYS <= set(d) and d["n_gpus"] == 1 and d["steps"] == 8 and d["scaling"] == "weak"
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert 0.3 < r["frac"] < 1.2 and r["traffic"] > 0
    assert d["gpu_launches"] >= 8 and d["value"] > 1e9
    e = d["e2e"]
    assert e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0 and 0 < e["value"] < d["value"]
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(d["clocks"])
    # the prune round is timed on every run, however few steps the timed loop has
    c = d["config"]
    assert c["prune_rounds_timed"] >= 3 and c["prune_round_ms"] > 0 and "workload" in c
    pr = c["prune_round"]
    assert abs(pr["prune_round_us"] - (pr["estimate_sparsity_us"] + pr["alloc_budgets_us"] + pr["rasr_prune_us"])) < 1e-6
    assert abs(pr["prune_amortised_us_per_step"] * pr["prune_interval"] - pr["prune_round_us"]) < 1e-6
    assert pr["rows_moved"] > 0 and pr["token_heads_after"] < pr["token_heads_before"]
    wp = r["with_amortised_prune"]
    assert wp["ms_per_step"] > c["attend_ms_per_step"] and 0.3 < wp["frac"] <= r["frac"]
    import bench
    assert set(c) == set(bench.CONFIG_KEYS)


@pytest.mark.gpu
def test_gpu_arm_on_a_quantised_cache():
    """The same line for `--kv fp8`: 264 algorithmic bytes per token-head, the per-layer launch mode included."""
    d = _run(["--kv", "fp8", "--steps", "8", "--warmup", "3", "--prep-rounds", "1", "--no-cpu-baseline"], timeout=900)
    assert BASE_KEYS <= set(d) and d["dtype"].startswith("fp8") and d["steps"] == 8
    r, c = d["roofline"], d["config"]
    assert abs(r["achieved"] - c["token_heads_per_step"] * 264 / (c["attend_ms_per_step"] * 1e-3) / 1e9) < 1e-6 * r["achieved"]
    assert 0.3 < r["frac"] < 1.2 and d["gpu_launches"] >= 8
    pl = c["per_layer_launch"]
    assert pl["ms_per_step"] > c["attend_ms_per_step"] and 0.05 < pl["frac"] < r["frac"]
    assert c["prune_rounds_timed"] >= 3 and d["e2e"]["h2d_bytes_per_step"] > 0
