"""Host-side pieces of bench.py that need no GPU: peak lookup, clock-sample parsing, CLI contract."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_peaks_come_from_the_measured_file_or_the_stated_fallback(tmp_path, monkeypatch):
    p = bench.load_peaks()
    assert p["source"] in ("measured", "fallback") and p["bf16_sustained"] > 100 and p["hbm_gbs"] > 1000
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.load_peaks() == dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")
    (tmp_path / "MEASURED_PEAKS.json").write_text(json.dumps(dict(hbm_gbs=1.0, bf16_tflops=2.0, bf16_tflops_sustained=3.0)))
    assert bench.load_peaks() == dict(hbm_gbs=1.0, bf16_burst=2.0, bf16_sustained=3.0, source="measured")


def test_clock_sampler_parses_nvidia_smi_lines():
    s = bench.ClockSampler(0)
    s.proc = type("P", (), {"terminate": lambda self: None, "wait": lambda self, timeout=None: 0, "kill": lambda self: None})()
    s.lines = ["0, 1300, 1965, 990.5, 0x0000000000000004, Not Active, Not Active, Not Active, Active",
               "0, 1250, 1965, 1001.0, 0x0000000000000004, Not Active, Not Active, Not Active, Active",
               "0, 1350, 1965, 980.0, 0x0000000000000000, Not Active, Not Active, Not Active, Not Active",
               "garbage"]
    c = s.stop()
    assert c["sm_mhz"] == 1300 and c["sm_max_mhz"] == 1965 and c["power_w_max"] == 1001.0 and c["samples"] == 3
    assert c["reasons"] == ["sw_power_cap"]
    s.lines = ["0, 900, 1965, 500, 0x8, Active, Not Active, Active, Not Active"]
    assert s.stop()["reasons"] == ["hw_slowdown", "sw_thermal_slowdown"]


def test_bench_refuses_to_run_without_a_gpu_instead_of_falling_back():
    import torch
    if torch.cuda.is_available():
        return
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "1"], capture_output=True, text=True)
    assert r.returncode != 0 and "no CPU fallback" in (r.stderr + r.stdout)
