"""bench.py from the command line, as far as that goes without a GPU: the reference arm (the fp64
oracle timed on the host cores) prints one JSON line with the agreed keys and the same `config` as the
product arm names; the product arm refuses to run without a CUDA device instead of falling back."""
import json
import os
import subprocess
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args):
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], cwd=ROOT, capture_output=True,
                          text=True, timeout=600)


def test_reference_arm_prints_one_json_line_with_the_agreed_keys():
    r = _run("--impl", "reference", "--steps", "1", "--warmup", "0")
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["value"] > 0 and d["ms_per_step"] > 0
    assert d["metric"] == "psa_attn_computed_tflops_at_75600_tokens" and d["unit"] == "TFLOP/s"
    assert d["n_gpus"] == 1 and d["steps"] == 1 and d["warmup"] == 0 and d["higher_is_better"] is True
    assert d["dtype"] == "f64" and d["data"] == "synthetic" and d["vs_baseline"] is None
    assert d["config"]["workload"] == "wan14b_720p" and "model" not in d["config"]
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["sample"] and cb["value"] == d["value"]
    e = d["e2e"]
    assert e["value"] == d["value"] and e["unit"] == d["unit"]
    assert e["h2d_bytes_per_step"] == 0 and e["d2h_bytes_per_step"] == 0
    # both arms name the workload with the same function
    sys.path.insert(0, ROOT)
    import bench
    from paper_2609_37001_b200 import workloads as WL
    assert set(d["config"].keys()) == set(bench.config_of(WL.workload("wan14b_720p")).keys())


def test_product_arm_refuses_to_run_without_a_gpu():
    if torch.cuda.is_available():
        return   # on a GPU machine the product arm is exercised by the GPU tests and the bench itself
    r = _run("--steps", "1", "--warmup", "0", "--quick")
    assert r.returncode != 0
    assert "no CPU fallback" in (r.stdout + r.stderr)
    assert not [l for l in r.stdout.splitlines() if l.startswith("{")]
