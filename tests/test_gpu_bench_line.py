"""bench.py on the device: one JSON line with the keys the benchmark contract names."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_has_the_contract_keys():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "5", "--warmup", "3"],
                         capture_output=True, text=True, cwd=ROOT, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks"):
        assert key in line, key
    assert line["n_gpus"] == 1 and line["steps"] == 5 and line["warmup"] >= 3
    assert line["config"]["workload"] == "tabular" and line["dtype"] == "bf16" and line["data"] == "synthetic"
    assert line["value"] > 0 and line["ms_per_step"] > 0
    roof = line["roofline"]
    assert roof["bound"] == "tensor" and roof["unit"] == "TFLOP/s" and roof["peak"] > 0
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9 and 0 < roof["frac"] < 1.2
    assert roof["traffic"] is None or roof["traffic"] > 0
    base = line["cpu_baseline"]
    assert base["kind"] == "oracle" and base["value"] > 0 and base["cores"] >= 1 and base["sample"]
    e2e = line["e2e"]
    assert e2e["value"] > 0 and e2e["h2d_bytes_per_step"] > 0 and e2e["d2h_bytes_per_step"] > 0
    assert e2e["value"] < line["value"]                       # host copies are inside its timed region
    assert line["gpu_launches"] > 0 and line["gpu_launches"] % line["steps"] == 0
    assert line["recomputed_clusters"] == 0                   # the timed path is the tensor-core kernel
    assert "sm_mhz" in line["clocks"] and "reasons" in line["clocks"]
    assert line["clocks"]["samples"] > 0 and line["clocks"]["sm_mhz"] > 0     # even with five timed steps
    # the clustering and selection kernels each against the roof that bounds them
    stages = line["stage_rooflines"]
    for name in ("gram", "transform", "split_levels", "split_tail", "permute_centroid"):
        st = stages[name]
        assert st["bound"] == "hbm" and st["ms"] > 0 and 0 < st["frac"] < 1.2
        assert abs(st["frac"] - st["achieved"] / st["peak"]) < 1e-9
    assert stages["score_select"]["bound"] == "alu" and 0 < stages["score_select"]["frac"] < 1.2
    assert stages["principal_components"]["ms"] > 0
    # the step's stages are made of these groups: their sum cannot be far below the clustering stage
    clustering = sum(stages[n]["ms"] for n in ("gram", "cholesky_factor", "principal_components", "transform",
                                               "split_levels", "split_tail", "permute_centroid"))
    assert clustering > 0.8 * line["stage_ms"]["cluster_qk"]
    # dense attention on the same GPU: torch's kernel and the library's own, the faster is the denominator
    dense = line["dense"]
    assert dense["library_ms"] > 0 and dense["fastest_ms"] == min(dense["library_ms"], dense["torch_sdpa_ms"])
    assert dense["speedup_vs_fastest_dense"] > 1.0
    sec = line["secondary"]
    assert sec["workload"] == "video480" and sec["head_dim"] == 128 and 0 < sec["roofline"]["frac"] < 1.2
    # the device's integer decisions for one head of the timed workload against the oracle
    dec = line["decisions_vs_oracle"]
    for side in ("queries", "keys"):
        rec = dec["sides"][side]
        assert rec["permutation_equals_float32_restatement"] is True
        assert rec["of_them_not_near_ties"] == 0 and rec["rows_in_another_cluster"] < 1e-3 * rec["rows"]
    assert dec["selection"]["lists_equal_float32_restatement"] is True
    assert dec["selection"]["of_them_not_near_ties"] == 0
