"""Host-side pieces of bench.py that need no GPU: the reference arm's JSON line (the oracle timed on the host cores)
and the clock sampler's bookkeeping."""
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line_with_the_contract_keys():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                          "--steps", "1", "--warmup", "1"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 1 and d["steps"] == 1 and d["warmup"] == 1
    assert d["unit"] == "instances/s" and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["value"] > 0 and abs(d["value"] - d["cpu_baseline"]["value"]) < 1e-9
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["value"] == d["value"] and d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert "workload" in d["config"] and "model" not in d["config"]


def test_reference_arm_does_nothing_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                          "--steps", "1", "--warmup", "1", "--gpus", "2"], capture_output=True, text=True, timeout=300,
                         cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    assert not [l for l in out.stdout.splitlines() if l.startswith("{")]


def test_clock_sampler_reports_the_samples_inside_the_timed_region():
    sys.path.insert(0, ROOT)
    import bench
    s = bench.ClockSampler(0)
    s.kind = "nvml"; s.smax = 1965.0
    t = time.perf_counter()
    s.samples = [(t - 3.0, 300.0, set()), (t - 1.0, 1900.0, {"sw_power_cap"}), (t - 0.9, 1950.0, set()),
                 (t - 0.8, 1965.0, set()), (t + 5.0, 400.0, {"hw_slowdown"})]
    s.t0, s.t1 = t - 1.5, t
    r = s.stop()
    assert r["samples"] == 3 and r["sm_mhz"] == 1950.0 and r["sm_max_mhz"] == 1965.0
    assert r["reasons"] == ["sw_power_cap"] and r["sampled"] == "during the timed region"
    # no sample inside: everything that was seen is reported, and the line says so
    s2 = bench.ClockSampler(0)
    s2.kind = "nvml"; s2.smax = 1965.0
    s2.samples = [(t - 3.0, 300.0, set()), (t + 5.0, 400.0, {"hw_slowdown"})]
    s2.t0, s2.t1 = t - 1.5, t
    r2 = s2.stop()
    assert r2["samples"] == 2 and r2["sampled"] == "around the timed region" and r2["reasons"] == ["hw_slowdown"]
    # neither NVML nor nvidia-smi
    assert bench.ClockSampler(0).stop()["sm_mhz"] is None
