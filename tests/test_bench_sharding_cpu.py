"""The multi-rank plumbing of bench.py on CPU: two gloo ranks shard the layers (every layer exactly once,
no data-path collective) and agree on the slowest rank's time.  No GPU involved."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.rank_world() == (rank, world, rank)
        mine = bench.shard_layers(32, rank, world)
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        slowest = bench.max_over_ranks(10.0 + 5.0 * rank)
        total = bench.sum_over_ranks(float(len(mine)))
        out.put((rank, gathered, slowest, total))
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_ranks_shard_layers_and_reduce_times():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = [out.get(timeout=90) for _ in range(world)]
    for p in procs:
        p.join(timeout=30)
        assert p.exitcode == 0
    for rank, gathered, slowest, total in results:
        layers = sorted(l for part in gathered for l in part)
        assert layers == list(range(32))                       # every layer once
        assert set(gathered[0]).isdisjoint(gathered[1])
        assert slowest == 15.0                                 # the max over ranks, on every rank
        assert total == 32.0


@pytest.mark.timeout(300)
def test_bench_starts_its_own_ranks_when_asked_for_several_gpus():
    """`python bench.py --gpus 2` outside a launcher must run as two ranks (here over gloo, plumbing only): rank 0 prints
    one JSON line that says n_gpus = 2 and shows every layer on exactly one rank."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["CUDA_VISIBLE_DEVICES"] = ""
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--plumbing-only"], env=env,
                         capture_output=True, text=True, timeout=280)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, res.stdout
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["backend"] == "gloo"
    assert sorted(l for part in line["layers_per_rank"] for l in part) == list(range(32))
    assert line["layers_total"] == 32.0 and line["slowest_rank_time"] == 15.0


def test_launcher_command_is_the_documented_one():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.launcher_command(4, ["--gpus", "4", "--steps", "7"], 29511)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29511"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "7"] and cmd[-5].endswith("bench.py")


def test_peak_kv_bytes_of_the_two_schedules():
    """Paragraph after Eq. 13: with budgets known beforehand a layer is compacted before the next one runs, so the
    peak is one full layer plus the compacted earlier ones; an online rule holds every layer uncompressed first."""
    import bench
    full = bench.kv_cache_bytes(1000, 2, 64)
    kept = [10.0, 20.0, 30.0]
    on = bench.kv_peak_bytes(3, 1000, kept, 2, 64, online=True)
    off = bench.kv_peak_bytes(3, 1000, kept, 2, 64, online=False)
    assert on == 3 * full
    assert off == full + bench.kv_cache_bytes(10, 2, 64) + bench.kv_cache_bytes(20, 2, 64)
    # nothing evicted: both schedules end up holding everything
    assert bench.kv_peak_bytes(3, 1000, [1000.0] * 3, 2, 64, online=False) == 3 * full


def test_single_process_helpers_are_no_ops():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.shard_layers(5, 0, 1) == [0, 1, 2, 3, 4]
    assert bench.max_over_ranks(3.5) == 3.5 and bench.sum_over_ranks(2.0) == 2.0


def test_kv_cache_accounting_of_the_32k_layer():
    """The paper's KV-size formula on the bench workload: a 32k-token LLaDA-shaped layer holds 536.9 MB of prompt keys
    and values in bf16, 4.19 MB once compacted to a mean budget of 256 tokens per head (a factor of 128)."""
    import bench
    full = bench.kv_cache_bytes(32768, 32, 128)
    kept = bench.kv_cache_bytes(256, 32, 128)
    assert full == 2 * 32768 * 32 * 128 * 2 == 536870912
    assert kept == 4194304 and full / kept == 128
    assert bench.kv_cache_bytes(100, 4, 64, elem_bytes=4) == 2 * 100 * 4 * 64 * 4
