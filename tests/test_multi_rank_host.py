"""The N > 1 path of bench.py on CPU: two gloo ranks shard the batch (replicas, no exchange step on
the data path) and reduce their device times with a max, as the GPU run does over NCCL."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import bench
    from paper_1907_01989_b200 import workloads as wl
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        batch = 3
        images = bench.shard_images(rank, batch)
        spec = wl.separable_block(batch)
        x = wl.make_input(spec, images=images)
        # rank r is 10 ms slower per unit of rank: the job time is the slowest rank's
        value, total_ms = bench.job_throughput(100.0 + 10.0 * rank, batch, 4, world, dist, "cpu")
        # every rank's shard, gathered only for the test (the data path itself has no collective)
        gathered = [None] * world
        dist.all_gather_object(gathered, (images, float(x.sum())))
        if rank == 0:
            out.put((value, total_ms, gathered))
    finally:
        dist.destroy_process_group()


def test_two_rank_sharding_and_max_reduction():
    from paper_1907_01989_b200 import workloads as wl
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    value, total_ms, gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert total_ms == 110.0                                   # max over ranks, not the mean
    assert abs(value - 2 * 3 * 4 / 0.110) < 1e-6               # all ranks' images over the slowest rank's time
    assert [g[0] for g in gathered] == [[0, 1, 2], [3, 4, 5]]  # disjoint, contiguous shards of the global batch
    # the shards are exactly the images a single process would draw for the global batch
    full = wl.make_input(wl.separable_block(6))
    assert np.isclose(gathered[0][1], float(full[:3].sum())) and np.isclose(gathered[1][1], float(full[3:].sum()))


def test_bench_gpus_2_starts_its_own_ranks():
    """`python bench.py --gpus 2` outside torchrun must start two ranks itself.  Run here without a GPU: each rank
    joins a gloo group, takes its shard and the ranks reduce with the timed run's own max-over-ranks code."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--host-check"], env=env, cwd=ROOT,
                       capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [json.loads(ln) for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                       # rank 0 alone prints
    line = lines[0]
    assert line["n_gpus"] == 2 and line["total_ms"] == 110.0
    assert abs(line["value"] - 2 * 3 * 4 / 0.110) < 1e-6
    assert [g[0] for g in line["shards"]] == [[0, 1, 2], [3, 4, 5]]


def test_bench_refuses_a_world_size_that_contradicts_gpus():
    import subprocess
    env = dict(os.environ, WORLD_SIZE="2", RANK="0")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--host-check"], env=env, cwd=ROOT,
                       capture_output=True, text=True, timeout=120)
    assert p.returncode != 0 and "WORLD_SIZE" in (p.stderr + p.stdout)


def test_single_rank_needs_no_process_group():
    import bench
    value, total_ms = bench.job_throughput(50.0, 8, 2, 1, None, "cpu")
    assert total_ms == 50.0 and abs(value - 8 * 2 / 0.05) < 1e-9


def test_clock_rows_are_filtered_by_the_timed_region():
    import bench
    rows = [(10.0, "t, 1200, 1965, 300, Not Active, Not Active, Not Active, Not Active"),
            (20.0, "t, 1950, 1965, 900, Not Active, Not Active, Not Active, Active"),
            (20.5, "t, 1900, 1965, 950, Not Active, Not Active, Not Active, Not Active"),
            (30.0, "t, 300, 1965, 100, Active, Not Active, Not Active, Not Active")]
    c = bench.summarize_clock_rows(rows, 19.0, 21.0)
    assert c["samples"] == 2 and c["sm_mhz"] == 1925.0 and c["sm_max_mhz"] == 1965.0 and c["reasons"] == ["sw_power_cap"]
    assert bench.summarize_clock_rows(rows)["samples"] == 4
