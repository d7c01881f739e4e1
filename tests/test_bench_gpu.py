"""bench.py on the GPU, tiny workload: one JSON line with every key the benchmark contract names, the same `config` object
as the reference arm, and a launch count that matches the library's own counter."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu


def test_gpu_arm_prints_the_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "tiny", "--steps", "5", "--warmup", "3",
                          "--condition-seconds", "0.2"], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.strip().splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["metric"] == "moe_layer_fwd_bwd_tokens_per_s" and d["unit"] == "tokens/s" and d["n_gpus"] == 1
    assert d["steps"] == 5 and d["warmup"] == 3 and d["higher_is_better"] is True and d["scaling"] == "weak"
    assert d["value"] > 0 and abs(d["value"] - 256 / (d["ms_per_step"] / 1e3)) <= 1e-6 * d["value"]
    assert d["dtype"] == "bf16" and d["data"] == "synthetic" and d["vs_baseline"] is None
    sys.path.insert(0, ROOT)
    import bench
    from paper_2608_00916_b200 import synth
    assert d["config"] == bench.workload_config("tiny", "train", synth.CONFIGS["tiny"][0], 1)
    rf = d["roofline"]
    assert rf["bound"] in ("tensor", "hbm") and rf["achieved"] > 0 and rf["peak"] > 0
    assert abs(rf["frac"] - rf["achieved"] / rf["peak"]) < 1e-9
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["value"] > 0 and cb["cores"] >= 1 and cb["sample"]
    e2e = d["e2e"]
    assert e2e["value"] > 0 and e2e["h2d_bytes_per_step"] == 2 * 256 * 256 * 2 and e2e["d2h_bytes_per_step"] > 0
    assert e2e["value"] != d["value"]
    assert "sm_mhz" in d["clocks"] and "reasons" in d["clocks"]
    assert d["graph_replay"]["ms_per_step"] > 0 and d["graph_replay"]["steps"] == 5
    rt = d["routing"]
    assert rt["rows_per_expert"]["mean"] == 256 * 2 / 8 and rt["empty_experts"] == 0 and len(rt["largest_five"]) == 5
    assert d["gpu_launches"] >= 5 * 10  # kernels of this library inside the timed region (5 steps)
