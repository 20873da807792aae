"""The multi-GPU arm of bench.py is "replicas only": every rank runs the whole layer on its own
batch, nothing is exchanged on the data path, and the job's throughput is all ranks' tokens over the
slowest rank's device time.  That host logic is checked here with two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from workloads import synth
    mine = [10.0 + 5.0 * rank, 30.0 - 7.0 * rank]          # rank 0: 10, 30; rank 1: 15, 23
    got = bench.max_over_ranks(mine, torch.device("cpu"), world)
    # every rank draws its own batch: different streams give different tokens
    a = synth.tokens(synth.WORKLOADS["c1"], stream=rank)
    q.put((rank, got, int(a[0, 0])))
    dist.destroy_process_group()


def test_slowest_rank_decides_and_batches_differ():
    world, port = 2, 29731
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == [15.0, 30.0] and res[1][1] == [15.0, 30.0]
    assert res[0][2] != res[1][2]


def test_job_value_is_all_ranks_tokens_over_the_slowest_time():
    import bench
    assert bench.job_tokens_per_s(1, 4096, 10, 5.0) == 4096 * 10 / 5e-3
    assert bench.job_tokens_per_s(8, 4096, 10, 5.0) == 8 * bench.job_tokens_per_s(1, 4096, 10, 5.0)
    assert bench.max_over_ranks([1.0, 2.0], torch.device("cpu"), 1) == [1.0, 2.0]


def test_gpus_flag_starts_the_replica_processes_itself():
    # `bench.py --gpus 2` with no launcher in the environment re-launches itself as two ranks (one per
    # GPU on a GPU machine).  Exercised here on the CPU with the reference arm, whose rank 0 alone works
    # and prints the line while rank 1 exits 0.
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference",
                        "--workload", "c1", "--steps", "1", "--warmup", "0"], capture_output=True, text=True,
                       env=env, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["config"]["workload"] == "c1"


def test_replica_command_is_one_rank_per_gpu_on_the_loopback_address():
    import bench
    cmd = bench.replica_command(4, ["--gpus", "4", "--steps", "7"], 29555)
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29555"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "7"]
