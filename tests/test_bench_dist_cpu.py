"""The multi-rank plumbing of bench.py on CPU: two gloo ranks agree on the slowest rank's time and
on the whole-job throughput. Rows are independent, so the data path itself has no collective."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, torch
    sys.path.insert(0, %r)
    os.environ["CUDA_VISIBLE_DEVICES"] = ""
    import bench
    rank, world, local = bench.dist_setup(2)
    assert world == 2 and rank == int(os.environ["RANK"])
    bench.barrier(world)
    mine = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    t = bench.max_over_ranks(mine, world, torch.device("cpu"))
    assert t == 15.0, t
    v = bench.aggregate(8192, world, t)
    assert abs(v - 2 * 8192 / 0.015) < 1e-6
    bench.barrier(world)
    import torch.distributed as dist
    dist.destroy_process_group()
    print("rank", rank, "ok")
""") % ROOT


def test_two_gloo_ranks_aggregate_like_the_bench(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29617", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o
        assert "ok" in o


def test_reference_arm_prints_one_json_line(tmp_path):
    import json
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "2", "--warmup", "1", "--oracle-rows", "16"], capture_output=True, text=True,
                         timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0


def test_reference_arm_of_the_hca_workloads(tmp_path):
    import json
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "hca-tiny",
                          "--steps", "2", "--warmup", "1", "--oracle-rows", "3"], capture_output=True, text=True,
                         timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["config"]["workload"] == "hca-tiny" and line["value"] > 0 and line["gpu_launches"] == 0
    # a rank other than 0 leaves without printing
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "hca-tiny",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300,
                         env=dict(os.environ, RANK="1", WORLD_SIZE="2"))
    assert out.returncode == 0 and out.stdout.strip() == ""
