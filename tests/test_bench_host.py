"""Host-side checks of bench.py: the reference arm's JSON line and the multi-rank
aggregation (N independent replicas, slowest rank's time) on two gloo ranks."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--workload", "cfg1", "--dtype", "f32", "--steps", "1", "--warmup", "1",
                          "--ref-macs", "2e5"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.strip().splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "TFLOP/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert d["config"]["workload"].startswith("cfg1")


_WORKER = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import torch, torch.distributed as dist
import bench
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
mine = 1.0 + 0.5 * rank                      # rank 1 is the slow replica
total = bench.max_over_ranks(mine, world, torch.device("cpu"))
assert total == 1.5, total
value = bench.replicas_value(3.0e12, world, total / 1)   # two replicas of 3 TFLOP each
assert abs(value - 2 * 3.0 / 1.5) < 1e-12, value
dist.barrier(); dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_replica_aggregation_on_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29533", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script), ROOT], env=dict(env, RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True)
             for r in range(2)]
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err
        assert "ok" in out


def test_alu_denominator_is_the_larger_of_the_measured_loop_and_the_unit_counts():
    """A register-only FMA loop measured under a power cap must not flatter the ALU-bound fractions:
    the denominator is never below 148 SMs x 128 (64) lanes x 2 x the sampled clock."""
    sys.path.insert(0, ROOT)
    import bench
    from workloads import F32, F64
    derived32 = 148 * 128 * 2 * 1965e6 / 1e12
    assert abs(bench.fma_peak(None, F32, 1965.0) - derived32) < 1e-9
    assert abs(bench.fma_peak(None, F64, 1965.0) - derived32 / 2) < 1e-9
    throttled = {"tflops": 53.8, "fp64": 25.8}
    assert bench.fma_peak(throttled, F32, 1965.0) == bench.fma_peak(None, F32, 1965.0)
    assert bench.fma_peak(throttled, F64, 1965.0) == bench.fma_peak(None, F64, 1965.0)
    high = {"tflops": 80.0, "fp64": 40.0}
    assert bench.fma_peak(high, F32, 1965.0) == 80.0 and bench.fma_peak(high, F64, 1965.0) == 40.0
    # a row sampled at a lower clock gets the measured loop if that is larger
    cool = {"tflops": 73.6, "fp64": 34.5}
    assert bench.fma_peak(cool, F32, 1500.0) == 73.6
