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


def test_roofline_model_arithmetic():
    """bench.place on hand-made rates: the ceiling is the slowest of the multiplier pipe, the ALU pipe,
    both pipes sharing the work, the issue slots and HBM; frac = ceiling time / measured time."""
    sys.path.insert(0, str(ROOT))
    import bench

    rates = {"r_wide": 30.0, "r_wide_isolated": 32.0, "r_imad": 64.0, "r_alu": 64.0, "r_issue": 128.0}
    w = bench.WORK["bias_context"]
    clocks = bench.unit_clocks(w, rates)
    assert abs(clocks["multiplier pipe"] - (w["wide"] / 30.0 + w["imad"] / 64.0)) < 1e-12
    assert abs(clocks["alu pipe"] - w["alu"] / 64.0) < 1e-12
    assert abs(clocks["both integer pipes"] - (w["wide"] * 64.0 / 30.0 + w["imad"] + w["alu"]) / 128.0) < 1e-12
    assert abs(clocks["issue slots"] - (w["wide"] + w["imad"] + w["alu"] + w["fp"]) / 128.0) < 1e-12
    units, mhz = 64 * 128256, 1965.0
    t_mul = clocks["multiplier pipe"] * units / (bench.SMS * mhz * 1e6)
    r = bench.place("bias_context", units, 4 * units, 2.0 * t_mul, rates, mhz, 6553.6)
    assert r["bound"] == "alu" and r["limiter"] == "multiplier pipe" and abs(r["frac"] - 0.5) < 1e-9
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-12 and r["frac_isolated"] < r["frac"]
    assert r["plain_eval"]["frac"] > r["frac"]                      # the plain count holds more products
    # a launch that moves so many bytes per unit that HBM is the ceiling
    r = bench.place("bias_context", units, 4000 * units, 1.0, rates, mhz, 6553.6)
    assert r["bound"] == "hbm" and abs(r["frac"] - 4000 * units / 6553.6e9) < 1e-9
    # least-work counts never exceed the plain-evaluation counts
    for kind, plain in bench.PLAIN_EVAL.items():
        least = bench.WORK[kind]
        assert least["wide"] <= plain["wide"] and least["wide"] + least["imad"] + least["alu"] <= \
            plain["wide"] + plain["imad"] + plain["alu"]


def test_clock_summary_uses_only_samples_inside_the_region():
    sys.path.insert(0, str(ROOT))
    import bench

    s = bench.ClockSampler.__new__(bench.ClockSampler)
    s.nv, s.max_mhz = object(), 1965.0
    s.samples = [(0.5, 1000.0, 0x1), (1.1, 1965.0, 0x0), (1.2, 1950.0, 0x4), (1.3, 1965.0, 0x0), (2.5, 300.0, 0x8)]
    out = s.summary(1.0, 2.0)
    assert out["samples"] == 3 and out["sm_mhz"] == 1965.0 and out["sm_min_mhz"] == 1950.0
    assert out["reasons"] == ["sw_power_cap"]                        # the slowdown outside the region is not reported
    assert s.summary(3.0, 4.0)["samples"] == 0 and s.summary(3.0, 4.0)["sm_mhz"] is None
