"""CPU: what `bench.py` promises without a GPU - the workload table carries the configurations' shapes and work, the
reference arm (the oracle on the host cores) prints one JSON line with the agreed keys, and a multi-GPU number is
refused on a box that does not have the GPUs."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _flops(spec):
    return sum(6.0 * spec["tokens"] * ly["d_in"] * ly["d_out"] for ly in spec["layers"])


def test_workload_table_matches_the_configurations():
    import bench
    w = bench.WORKLOADS
    assert bench.HEADLINE == "block_16384tok"
    # forward + input gradient + weight gradient of every layer: 6 l m n
    assert _flops(w["qproj_4096tok"]) == pytest.approx(0.412e12, rel=2e-3)
    assert _flops(w["ffn_8192tok"]) == pytest.approx(8.66e12, rel=2e-3)
    assert _flops(w["block_16384tok"]) == pytest.approx(21.44e12, rel=2e-3)
    for k in (0, 16, 64, 256):
        spec = w["proj70b_16384tok_k%d" % k]
        assert spec["k"] == k and spec["rank"] == 64 and _flops(spec) == pytest.approx(23.09e12, rel=2e-3)
    block = w["block_16384tok"]
    assert [ly["name"] for ly in block["layers"]] == ["q", "k", "v", "o", "gate", "up", "down"]
    assert len({ly["x"] for ly in block["layers"]}) == 4                # q/k/v and gate/up share their input
    assert all(spec["k"] % 4 == 0 for spec in w.values())


def test_reference_arm_prints_the_agreed_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "split_fp4_linear_fwd_bwd_effective_tflops" and d["unit"] == "TFLOP/s"
    assert d["n_gpus"] == 1 and d["steps"] == 1 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["dtype"] == "f64" and d["data"] == "synthetic" and "workload" in d["config"]
    assert d["value"] > 0 and d["ms_per_step"] > 0
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == d["value"] and cb["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["gpu_launches"] == 0


def test_a_multi_gpu_number_is_refused_without_the_gpus():
    import torch
    if torch.cuda.device_count() >= 2:
        pytest.skip("two GPUs present")
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"], capture_output=True, text=True,
                       timeout=300, cwd=ROOT, env=env)
    assert r.returncode == 2 and "refusing" in r.stderr
    assert not [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
