"""The benchmark's baseline arm (the CPU oracle on a bounded sample) prints one JSON line with the agreed keys.
CPU only; the GPU arm is exercised on a GPU machine."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line_with_the_agreed_keys():
    import time
    t0 = time.perf_counter()
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "600", "--warmup", "3"],
                       capture_output=True, text=True, timeout=600, cwd=ROOT)
    p_seconds = time.perf_counter() - t0
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["metric"] == "validated_bytes_per_second" and j["unit"] == "GB/s"
    assert j["n_gpus"] == 1 and j["steps"] == 600 and j["warmup"] == 3 and j["higher_is_better"] is True
    assert j["value"] > 0 and j["ms_per_step"] > 0 and j["vs_baseline"] is None and j["data"] == "synthetic"
    assert j["config"]["workload"] == "config4"
    cb = j["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] == 1 and cb["value"] == j["value"] and cb["sample"]
    e = j["e2e"]
    assert e["value"] == j["value"] and e["unit"] == "GB/s" and e["h2d_bytes_per_step"] == 0 and e["d2h_bytes_per_step"] == 0
    # the same config keys as the GPU arm's line, and a step time that is what one step of this run really took
    assert set(j["config"]) == {"workload", "what", "step", "algorithmic_bytes_per_step", "l2", "replicas"}
    assert j["config"]["algorithmic_bytes_per_step"] == 17 * (1 << 30)
    assert j["ms_per_step"] * j["steps"] < 1e3 * p_seconds and j["full_step_ms_estimate"] > j["ms_per_step"]


def test_gpus_n_without_a_launcher_re_executes_under_torch_distributed_run():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.torchrun_command(4, ["--gpus", "4", "--steps", "7"])
    assert cmd[0] == sys.executable and cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--nnodes=1" in cmd and cmd[cmd.index("--nproc-per-node") + 1] == "4"
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and int(cmd[cmd.index("--master-port") + 1]) > 0
    assert cmd[-5] == os.path.join(ROOT, "bench.py") and cmd[-4:] == ["--gpus", "4", "--steps", "7"]


def test_a_rank_count_that_contradicts_gpus_is_refused():
    env = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "4", "--steps", "1"],
                       capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert p.returncode != 0 and p.stdout.strip() == ""


def test_ranks_other_than_zero_of_the_reference_arm_do_no_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "2"],
                       capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert p.returncode == 0 and p.stdout.strip() == ""


import pytest


@pytest.mark.gpu
def test_gpu_arm_prints_one_json_line_with_roofline_e2e_and_cpu_baseline():
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "config2", "--steps", "20", "--warmup", "3"],
                       capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [l for l in p.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["metric"] == "validated_bytes_per_second" and j["unit"] == "GB/s" and j["n_gpus"] == 1 and j["steps"] == 20
    assert j["value"] > 0 and j["scaling"] == "weak" and j["dtype"] == "f32" and j["config"]["workload"] == "config2"
    assert j["gpu_launches"] >= 4 * 20                      # per step: gen, pass 1, pass 2 with the verdicts, fitness (the plan is reused)
    assert j["n_gpus_requested"] == 1 and j["per_config"] is None          # the other populations ride on the default run only
    m = j["cpu_baseline_all_cores"]
    assert m["cores"] >= 1 and m["value"] > 0 and "disjoint" in m["kind"]
    r = j["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert r["frac_of_datasheet"] < r["frac"] and r["datasheet_peak"] == 7700.0
    assert r["frac_alone"] > 0 and r["kernel_ms_alone"] > 0              # the kernel with nothing beside it, after the timed region
    gen = j["roofline_generator"]
    assert gen["bound"] == "alu" and 0 < gen["frac"] < 1.2 and abs(gen["frac"] - gen["achieved"] / gen["peak"]) < 1e-9
    assert j["streams"].startswith("evo_gen_inputs on a second stream")
    e = j["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] >= j["config"]["algorithmic_bytes_per_step"] and e["d2h_bytes_per_step"] > 0
    c = j["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] == 1 and c["value"] > 0 and c["sample"]
    assert set(j["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
