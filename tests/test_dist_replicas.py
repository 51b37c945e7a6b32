"""The multi-GPU mode of the benchmark is data-parallel replicas: every rank runs its own block,
and only the step time crosses ranks (max over ranks after a barrier).  These tests run that host
logic as two gloo ranks on CPU."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, {root!r})
    import torch.distributed as dist
    import bench
    rank, world, local = bench.dist_info()
    dist.init_process_group("gloo")
    bench.barrier(world)
    # each rank reports a different time; every rank must get the slowest one
    got = bench.reduce_max(10.0 + 5.0 * rank, world)
    # whole-job throughput = units of all ranks / the slowest rank's time
    units = 1000 * world
    print(json.dumps({{"rank": rank, "world": world, "max": got, "value": units / got}}))
    bench.barrier(world)
    dist.destroy_process_group()
""")


def _run_two_ranks(tmp_path, port):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err[-2000:]
        outs.append(out.strip().splitlines()[-1])
    return outs


def test_two_ranks_agree_on_the_slowest_time(tmp_path):
    import json
    outs = [json.loads(o) for o in _run_two_ranks(tmp_path, 29731)]
    assert sorted(o["rank"] for o in outs) == [0, 1]
    for o in outs:
        assert o["world"] == 2
        assert o["max"] == 15.0                    # rank 1's time
        assert abs(o["value"] - 2000 / 15.0) < 1e-9


def test_reference_arm_runs_on_rank_zero_only(tmp_path):
    # `bench.py --impl reference` under a 2-rank launch: rank 0 prints the line, rank 1 exits 0 silently
    outs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT="29732")
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                            "--workload", "single_f32", "--steps", "1", "--warmup", "0"],
                           env=env, capture_output=True, text=True, timeout=300)
        assert r.returncode == 0, r.stderr[-2000:]
        outs.append(r.stdout.strip())
    import json
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0
    assert outs[1] == ""
