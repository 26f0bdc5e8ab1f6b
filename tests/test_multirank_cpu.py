"""The N > 1 path of the benchmark on CPU: two gloo ranks, each an independent replica; the only exchange is a
barrier and the maximum of the per-rank timings, from which rank 0 computes the whole-job throughput."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    dist.barrier()
    ms = [10.0, 30.0][rank]                       # rank 1 is the slow one
    red = bench.max_over_ranks([ms, ms * 2], world)
    value = bench.whole_job_value(1000, 5, world, red[0])
    name, scale = bench.pick_workload("tiny", world)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"red": red, "value": value, "workload": name}))
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_reduce_to_the_slowest_rank(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29731", str(script)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert res["red"] == [30.0, 60.0]                         # max over ranks
    assert abs(res["value"] - 1000 * 2 * 5 / 0.030) < 1e-6    # both replicas' inputs in the slowest rank's time
    assert res["workload"] == "tiny"


def test_single_rank_helpers():
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1) == [1.5, 2.5]
    assert abs(bench.whole_job_value(16384, 100, 1, 64.6) - 16384 * 100 / 0.0646) < 1e-3


def test_reference_arm_under_two_ranks_runs_on_rank_zero_alone():
    """`bench.py --impl reference` launched as two ranks: rank 0 times the oracle and prints the one JSON line, the
    other rank leaves with exit code 0 and prints nothing; neither loads the CUDA library."""
    import json
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29733", os.path.join(ROOT, "bench.py"),
                          "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "3", "--workload", "tiny"],
                         capture_output=True, text=True, env=env, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    res = json.loads(lines[0])
    assert res["impl"] == "reference" and res["n_gpus"] == 2 and res["value"] > 0
    assert res["cpu_baseline"]["kind"] == "oracle" and res["e2e"]["h2d_bytes_per_step"] == 0
