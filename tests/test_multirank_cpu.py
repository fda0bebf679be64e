"""The N > 1 path of the benchmark is "replicas only": ranks run independently and every reported time is
the maximum over the ranks.  The cross-rank logic is exercised here with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    vals = bench.max_over_ranks([100.0 + rank, 5.0 - rank, 7.0], torch.device("cpu"), world)
    dist.barrier()
    out.put((rank, vals))
    dist.destroy_process_group()


def test_times_are_the_maximum_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 500
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got[0] == got[1] == [101.0, 5.0, 7.0]


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0], torch.device("cpu"), 1) == [3.0, 4.0]


def test_reference_arm_prints_only_on_rank_0():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--gpus", "2"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_gpus_flag_starts_the_replica_processes_itself():
    """`bench.py --gpus 2` run plainly (no launcher's environment) starts two ranks, which rendezvous, take the
    maximum over the ranks, and report n_gpus = 2: here on CPU with gloo through the plumbing-check mode."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--plumbing-check"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(x) for x in r.stdout.splitlines() if x.startswith("{")]
    assert len(lines) == 1
    assert lines[0]["n_gpus"] == 2 and lines[0]["max_over_ranks"] == [101.0, 5.0]


def test_workload_tables_are_consistent():
    sys.path.insert(0, ROOT)
    import bench
    w = dict(bench.WORKLOADS["7b_hbm_1800f"], name="7b_hbm_1800f")
    ab = bench.algorithmic_bytes(w)
    assert ab["kv"] == 28 * 72 * 401408 and ab["reps"] == 28 * 1800 * 512 * 4
    assert abs(ab["total"] - 925.3e6) < 1e6
    assert abs(bench.attention_flops(w) - 181.3e9) < 1e9
    # the line the reference arm prints is valid JSON with the contract's keys (short run)
    assert {"7b_hbm_1800f", "7b_offload_10800f", "7b_stream_batch16", "72b_offload_1800f"} <= set(bench.WORKLOADS)
