"""bench.py --tables: the markdown tables are a pure function of a stored JSON line (no GPU)."""
import json
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parents[1]


def stored_line():
    clocks = {"sm_mhz": 1965.0, "sm_max_mhz": 1965, "reasons": [], "samples": 12}
    return {
        "metric": "verify_step_latency_ms", "value": 0.0627, "unit": "ms",
        "config": {"workload": "cfg1 step"},
        "latency": {"median_ms": 0.0627, "p10_ms": 0.0626, "p90_ms": 0.0628, "eager_median_ms": 0.0662},
        "clocks": clocks, "e2e": {"value": 3.09, "unit": "ms"},
        "kernels": {
            "attention": {"ms": 0.0223, "tflops": 770.0, "frac_of_measured": 0.464, "frac_of_nominal_2250": 0.342},
            "verify": {"ms": 0.0387, "gbs": 3348.0, "frac_of_measured": 0.510, "frac_of_nominal_8000": 0.419},
        },
        "other_configs": [
            {"name": "sweep N=4096", "op": "dd_bidir_attention", "ms": 1.0426, "p10": 0.9514, "p90": 1.0472, "bound": "tensor",
             "tflops": 1055.0, "frac_of_measured_burst": 0.635, "frac_of_measured_sustained": 0.760,
             "frac_of_nominal_2250": 0.469, "clocks": dict(clocks, sm_mhz=1747.0, reasons=["sw_power_cap"])},
            {"name": "cfg2 batched serving CONF", "op": "dd_verify", "ms": 0.1263, "p10": 0.1224, "p90": 0.1264, "bound": "hbm",
             "gbs": 5174.0, "frac_of_measured_hbm": 0.789, "frac_of_nominal_8000": 0.647, "clocks": clocks},
        ],
    }


def test_tables_from_a_stored_line(tmp_path):
    path = tmp_path / "line.json"
    # the stored file may hold other output before the line: the last line that is JSON counts
    path.write_text("warming up\n" + json.dumps(stored_line()) + "\n")
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--tables", str(path)], capture_output=True, text=True,
                         cwd=ROOT, timeout=120)
    assert out.returncode == 0, out.stderr
    text = out.stdout
    assert "62.70 us per step" in text and "eager launches 66.20 us" in text
    assert "| attention | 22.30 | 770 TFLOP/s | 0.464 (burst) | 0.342 of 2250 |" in text
    assert "| verify | 38.70 | 3348 GB/s | 0.510 | 0.419 of 8000 |" in text
    assert "| sweep N=4096 | dd_bidir_attention | 1042.6 | 951.4 / 1047.2 | 1055 TFLOP/s | 0.635 burst, 0.760 sustained | 0.469 | 1747.0 (sw_power_cap) |" in text
    assert "| cfg2 batched serving CONF | dd_verify | 126.3 | 122.4 / 126.4 | 5174 GB/s | 0.789 | 0.647 | 1965.0 (none) |" in text
