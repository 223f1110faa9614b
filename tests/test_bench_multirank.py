"""The benchmark's N > 1 logic (max-over-ranks timing, rank-0 reporting) on two gloo ranks on CPU."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank = dist.get_rank()
    t = bench.aggregate_max(10.0 + 5.0 * rank, torch.device("cpu"))      # rank 1 is the slow one
    n = 1000
    if rank == 0:
        print(json.dumps({"t": t, "value": dist.get_world_size() * n / (t * 1e-3)}))
    dist.destroy_process_group()
""") % ROOT


def test_two_rank_timing_takes_the_max_over_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29517", str(script)],
                         capture_output=True, text=True, timeout=240, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    j = json.loads(line)
    assert j["t"] == 15.0
    assert abs(j["value"] - 2 * 1000 / 15e-3) < 1e-6


def test_reference_arm_prints_one_json_line_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "small",
                          "--steps", "1"], capture_output=True, text=True, timeout=240, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "small",
                          "--steps", "1"], capture_output=True, text=True, timeout=240, env=env)
    j = json.loads(out.stdout.strip().splitlines()[-1])
    assert j["impl"] == "reference" and j["cpu_baseline"]["kind"] == "oracle" and j["value"] > 0
    assert j["e2e"]["h2d_bytes_per_step"] == 0


def test_clock_sampler_summary_separates_load_from_idle_and_the_two_power_readings():
    """The summary of the nvidia-smi samples: median clock, throttle reasons, power as the mean of the samples taken
    under load, the averaged and the unaveraged reading kept apart, and nothing when there are no samples."""
    sys.path.insert(0, ROOT) if ROOT not in sys.path else None
    import bench
    s = bench.ClockSampler.__new__(bench.ClockSampler)
    idle = ["1965", "1965", "190.0", "Not Active", "Not Active", "Not Active", "Not Active"]
    load = ["1260", "1965", "900.0", "Not Active", "Not Active", "Not Active", "Active"]
    s.rows = [idle, load, load, load]
    out = s.summary()
    assert out["sm_mhz"] == 1260.0 and out["sm_max_mhz"] == 1965.0 and out["reasons"] == ["sw_power_cap"]
    assert out["watts"] == 900.0 and out["watts_instant"] is None and out["samples"] == 4
    s.rows = [idle + ["200.0"], load + ["1010.0"], load + ["990.0"]]
    out = s.summary()
    assert out["watts"] == 900.0 and out["watts_instant"] == 1000.0
    s.rows = []
    out = s.summary()
    assert out["sm_mhz"] is None and out["watts"] is None and out["watts_instant"] is None and out["reasons"] == []
