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


def test_bench_spawns_its_own_ranks_when_no_launcher_did(tmp_path):
    """`bench.py --gpus 2` without torchrun: spawn_ranks starts two processes whose environment is enough for a
    gloo rendezvous, and fails as a whole when one rank fails."""
    import bench
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    clean = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT")}
    old = dict(os.environ)
    os.environ.clear()
    os.environ.update(clean)
    try:
        assert bench.spawn_ranks(2, [sys.executable, str(script)], timeout=120) == 0
        bad = tmp_path / "bad.py"
        bad.write_text("import os, sys, time\nif os.environ['RANK'] == '1':\n    sys.exit(3)\ntime.sleep(60)\n")
        assert bench.spawn_ranks(2, [sys.executable, str(bad)], timeout=120) == 3     # rank 0 is not left sleeping
    finally:
        os.environ.clear()
        os.environ.update(old)
    # the command line a user types: the reference arm needs no GPU; rank 0 prints the one line with n_gpus = 2
    import json
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference",
                          "--workload", "tiny", "--steps", "1", "--warmup", "0", "--oracle-rows", "8"],
                         capture_output=True, text=True, timeout=300, env=clean)
    assert out.returncode == 0, out.stderr
    lines = [ln for ln in out.stdout.strip().splitlines() if ln.startswith("{")]
    assert len(lines) == 1 and json.loads(lines[0])["n_gpus"] == 2
    # our own arm refuses to pretend: more GPUs asked for than visible is an error, not an n_gpus = 1 line
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--workload", "tiny"],
                         capture_output=True, text=True, timeout=300, env=dict(clean, CUDA_VISIBLE_DEVICES=""))
    assert out.returncode != 0 and "--gpus 2" in out.stderr and out.stdout.strip() == ""


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
