"""The N > 1 path of the benchmark on CPU: two gloo ranks, no GPU.

The convolution path shards over images with no collective (replicas), so what N > 1 adds is only the
aggregation: the step time is the maximum over ranks and the job's throughput counts every replica's work.
"""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%%s" %% os.environ["MASTER_PORT"], rank=rank, world_size=world)
    mine = [10.0 + 5.0 * rank, 40.0 - 3.0 * rank]          # rank 0: (10, 40); rank 1: (15, 37)
    got = bench.max_over_ranks(mine, world, "cpu")
    dist.barrier()
    print(json.dumps({"rank": rank, "got": got, "value": bench.whole_job_gflops(10**9, world, got[0])}))
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_take_the_max_and_count_both_replicas(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = str(29500 + os.getpid() % 2000)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=port)
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        o, e = p.communicate(timeout=180)
        assert p.returncode == 0, e
        outs.append(json.loads(o.strip().splitlines()[-1]))
    for o in outs:
        assert o["got"] == [15.0, 40.0]                       # max over ranks of each entry
        assert abs(o["value"] - 2 * 1e9 / 15e-3 / 1e9) < 1e-9   # two replicas' FLOPs over the slowest rank's time


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1, "cpu") == [1.5, 2.5]
    assert bench.whole_job_gflops(43065365760, 1, 0.2) == 43065365760 / 0.2e-3 / 1e9
