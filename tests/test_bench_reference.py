"""The reference arm of the benchmark (the CPU oracle timed on the host cores) prints one JSON line with the
contract's keys; no GPU is involved."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "1",
                          "--config", "1"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "GB/s" and d["higher_is_better"] is True and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"].startswith("config 1")


def test_other_ranks_of_the_reference_arm_do_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_reference_arm_times_exactly_the_requested_steps_and_labels_the_extrapolation():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "3", "--warmup", "1",
                          "--config", "1"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    d = json.loads(out.stdout.strip())
    assert d["steps"] == 3 and d["cpu_baseline"]["sample"].startswith("3 steps")
    # config 1 has one sequence: the sample is the whole batch and the extrapolation changes nothing
    assert d["ms_per_step_extrapolated_full_batch"] == d["ms_per_step"] > 0


def test_measured_peak_falls_back_when_the_file_is_missing(tmp_path):
    sys.path.insert(0, ROOT)
    import bench
    peak, src = bench.measured_peak(str(tmp_path / "absent.json"))
    assert peak == bench.FALLBACK_HBM_GBS and src.startswith("fallback")
    bad = tmp_path / "bad.json"
    bad.write_text("{not json")
    assert bench.measured_peak(str(bad))[0] == bench.FALLBACK_HBM_GBS
    good = tmp_path / "good.json"
    good.write_text(json.dumps({"hbm_gbs": 6000.5}))
    assert bench.measured_peak(str(good)) == (6000.5, "measured (MEASURED_PEAKS.json, stream copy)")
