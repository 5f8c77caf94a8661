"""Host-side logic of the benchmark: row sharding and the max-over-ranks reduction, on two gloo ranks."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def test_shard_rows_partitions_exactly():
    import bench
    for M, world in ((4096, 2), (4097, 2), (10, 4), (3, 8), (0, 2)):
        blocks = [bench.shard_rows(M, r, world) for r in range(world)]
        assert blocks[0][0] == 0 and blocks[-1][1] == M
        for (a, b), (c, d) in zip(blocks, blocks[1:]):
            assert b == c and b >= a
        sizes = [b - a for a, b in blocks]
        assert max(sizes) - min(sizes) <= 1


def test_flop_and_byte_model():
    import bench
    f1, f3 = bench.layer_flops(4096, 4096, 14336)
    assert f1 == 2 * 4096 ** 3 and f3 == 2 * 4096 * 4096 * 14336
    byts = bench.layer_bytes(4096, 4096, 14336, "mxfp4")
    assert abs(byts - (2 * 4096 * 4096 * 2 + 14336 * 4096 * (0.5 + 1 / 32) + 4 * 4096 * 14336)) < 1


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    lo, hi = bench.shard_rows(1001, rank, world)
    t = bench.reduce_max_time(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
    rows = torch.tensor([hi - lo], dtype=torch.int64)
    dist.all_reduce(rows)
    out[rank] = (t, int(rows.item()))
    dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_gloo_ranks_agree_on_the_slowest_time():
    world, port = 2, 29500 + os.getpid() % 2000
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0] == out[1] == (15.0, 1001)


@pytest.mark.timeout(180)
def test_gpus_flag_spawns_that_many_ranks():
    """`bench.py --gpus 2` without a launcher starts two ranks itself (here on gloo, no GPU work) and reports n_gpus = 2;
    asked for more GPUs than the machine has, the GPU arm refuses instead of running on fewer."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--plumbing-only", "--workload", "cfg1"],
                       capture_output=True, text=True, env=env, timeout=170)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads([ln for ln in r.stdout.splitlines() if ln.startswith("{")][-1])
    assert line["n_gpus"] == 2 and line["ms_slowest_rank"] == 2.0 and line["rows_total"] == 2 * 2048
    if torch.cuda.device_count() < 64:
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "64", "--steps", "1"],
                           capture_output=True, text=True, env=env, timeout=170)
        assert r.returncode == 2 and "GPU(s) visible" in r.stderr


def test_regime_follows_the_sampled_clock():
    import bench
    full = dict(sm_mhz=1965.0, sm_max_mhz=1965.0, reasons=[])
    capped = dict(sm_mhz=1400.0, sm_max_mhz=1965.0, reasons=["sw_power_cap"])
    slow = dict(sm_mhz=1400.0, sm_max_mhz=1965.0, reasons=[])
    assert bench.pick_regime(full, 4.0) == "burst" and bench.pick_regime(full, 2000.0) == "burst"
    assert bench.pick_regime(capped, 4.0) == "sustained" and bench.pick_regime(slow, 2000.0) == "sustained"
    assert bench.pick_regime(dict(sm_mhz=None, sm_max_mhz=None, reasons=[]), 2000.0) == "burst"
