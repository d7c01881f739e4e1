"""The reference arm of bench.py (the CPU oracle timed as it stands) runs without a GPU and prints one JSON line with the
keys the benchmark contract names; the algorithmic-work table covers every stage the library times."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_the_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.strip().splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "moe_layer_fwd_bwd_tokens_per_s" and d["unit"] == "tokens/s"
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["steps"] == 2 and d["warmup"] == 1
    assert d["value"] > 0 and d["ms_per_step"] > 0 and d["config"]["workload"] == "tiny"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    # the same `config` object as the GPU arm prints for the same arguments
    sys.path.insert(0, ROOT)
    import bench
    from paper_2608_00916_b200 import synth
    assert d["config"] == bench.workload_config("tiny", "train", synth.CONFIGS["tiny"][0], 1)


def test_reference_arm_on_other_ranks_does_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--gpus", "2", "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=120,
                         cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_stage_work_covers_every_timed_stage():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2608_00916_b200 import synth
    from paper_2608_00916_b200.binding import STAGE_NAMES
    shape = synth.CONFIGS["qwen"][0]
    work = bench.stage_work(shape)
    assert set(work) == set(STAGE_NAMES)
    R = shape.T * shape.k
    gemm = sum(v for k, (kind, v) in work.items() if kind == "tensor")
    assert gemm == 18 * R * shape.d * shape.f  # 6 forward + 12 backward flops per routed row and weight element
    assert all(v > 0 for _, v in work.values())
