"""The JSON line of bench.py: the reference arm (the oracle, CPU only) here, the GPU arm on a
B200.  Checks the keys and the internal consistency of the numbers, not their size."""
import json
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config", "e2e"}


def _run(*args):
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), *args], cwd=ROOT, capture_output=True, text=True,
                         timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    return json.loads(lines[0])


def test_reference_arm_prints_the_contract_line():
    d = _run("--impl", "reference", "--steps", "2", "--warmup", "1")
    assert BASE_KEYS <= set(d) and d["impl"] == "reference"
    assert d["metric"] == "sbw_bias_throughput" and d["unit"] == "Gelem/s" and d["higher_is_better"] is True
    assert d["steps"] == 2 and d["warmup"] == 1 and d["vs_baseline"] is None and d["data"] == "synthetic"
    assert "workload" in d["config"] and "model" not in d["config"]
    assert set(d["config"]) == {"workload", "B", "V", "scheme", "gamma", "delta", "l2"}    # same keys as the GPU arm
    assert d["value"] > 0 and abs(d["value"] - 64 * 128256 / (d["ms_per_step"] * 1e-3) / 1e9) < 1e-6 * d["value"]
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["sample"] and cb["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


@pytest.mark.gpu
def test_gpu_arm_prints_the_contract_line():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    d = _run("--steps", "64", "--warmup", "3")
    assert BASE_KEYS | {"clocks", "gpu_launches", "roofline", "cpu_baseline", "roofline_detect", "cpu_baseline_detect",
                        "roofline_sample", "replays", "detect_tokens_per_s"} <= set(d) and "impl" not in d
    assert d["n_gpus"] == 1 and d["steps"] == 64 and d["warmup"] == 3 and d["gpu_launches"] == 64 * d["replays"]
    assert d["timed_region_s"] >= 0.25 and d["clocks"]["samples"] >= 50      # clocks sampled inside the region
    assert set(d["config"]) == {"workload", "B", "V", "scheme", "gamma", "delta", "l2"}
    assert d["dtype"] == "bf16" and d["scaling"] == "weak" and d["vs_baseline"] is None
    elems = 64 * 128256
    assert abs(d["value"] - elems / (d["ms_per_step"] * 1e-3) / 1e9) < 1e-6 * d["value"]
    r = d["roofline"]
    assert r["bound"] in ("alu", "hbm", "tensor") and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert 0.3 < r["frac"] <= 1.05 and (r["traffic"] is None or r["traffic"] > 0)
    assert "measured in this run" in r["peak_source"]
    for key in ("roofline_detect", "roofline_detect_selfsalt", "roofline_sample"):      # per-pipe placement of
        q = d[key]                                                                     # the other kernels
        assert q["bound"] in ("alu", "hbm") and 0.2 < q["frac"] <= 1.05 and abs(q["frac"] - q["achieved"] / q["peak"]) < 1e-9
    assert abs(d["detect_tokens_per_s"] - d["roofline_detect"]["tokens_per_s"]) < 1
    cd = d["cpu_baseline_detect"]
    assert cd["kind"] == "oracle" and cd["unit"] == "tokens/s" and 0 < cd["value"] < d["detect_tokens_per_s"]
    for name, e in d["extra"].items():
        if isinstance(e, dict) and "frac" in e:
            assert e["frac"] <= 1.05, (name, e["frac"])
    e = d["e2e"]
    assert e["h2d_bytes_per_step"] >= elems * 2 and e["d2h_bytes_per_step"] == elems * 2
    assert 0 < e["value"] < d["value"]                         # the copies are inside that timed region
    c = d["clocks"]
    assert c["sm_mhz"] > 0 and c["sm_max_mhz"] >= c["sm_mhz"] and isinstance(c["reasons"], list)
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and 0 < cb["value"] < d["value"]
