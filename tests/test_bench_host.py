"""CPU-side checks of bench.py: the reference arm prints a well-formed JSON line, and the multi-rank
aggregation (max time over ranks, sum of work) runs with two gloo processes."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_the_contract_line():
    out = subprocess.check_output([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                                   "tiny", "--steps", "2", "--warmup", "3", "--ref-blocks", "16"], text=True, timeout=600)
    line = json.loads(out.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "TFLOP/s" and line["value"] > 0
    assert line["steps"] == 2 and line["warmup"] == 3 and line["higher_is_better"] is True
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"] == {"value": line["value"], "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert "tiny" in line["config"]["workload"] and line["dtype"] == "f64" and line["vs_baseline"] is None


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 1 is slower: the job time is its time; the work is the sum of both ranks' work
    ms, tflops, w = bench.aggregate_over_ranks(2.0 if rank == 0 else 5.0, 1e12 * (rank + 1), dist, device="cpu")
    reqs = [bench.make_request("tiny", r) for r in (0, 1)]
    q.put((rank, ms, tflops, w, reqs[0].qkv_seed != reqs[1].qkv_seed))
    dist.barrier()
    dist.destroy_process_group()


def _shard_rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    from paper_2609_25869_b200 import shard
    dist.init_process_group("gloo", rank=rank, world_size=world)
    H = 5  # uneven: rank 0 gets 3 heads, rank 1 gets 2
    lo, hi = shard.head_range(H, rank, world)
    full = torch.arange(H * 4 * 3, dtype=torch.float32).reshape(H, 4, 3)
    got = shard.all_gather_heads(full[lo:hi].clone(), H, dist)
    q.put((rank, (lo, hi), bool(torch.equal(got, full))))
    dist.barrier()
    dist.destroy_process_group()


def test_head_sharding_ranges_and_gather_with_gloo():
    """Head-sharded driver, host side: ranges partition the heads for every (H, world), and the padded all-gather
    puts uneven shards back together on both ranks."""
    sys.path.insert(0, ROOT)
    from paper_2609_25869_b200 import shard
    for H in range(0, 40):
        for world in range(1, 10):
            rs = shard.head_ranges(H, world)
            assert rs[0][0] == 0 and rs[-1][1] == H
            assert all(a[1] == b[0] for a, b in zip(rs[:-1], rs[1:]))
            sizes = [hi - lo for lo, hi in rs]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_shard_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, (0, 3), True), (1, (3, 5), True)]


def test_two_rank_aggregation_with_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, tflops, w, distinct in res:
        assert w == 2 and ms == 5.0 and distinct          # max over ranks; each rank has its own inputs
        assert abs(tflops - (1e12 + 2e12) / 5e-3 / 1e12) < 1e-9
