"""The N>1 host logic on CPU: two gloo ranks, head sharding with no collective on the data path,
step time reduced as the max over ranks."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2607_24377_b200 import sharding
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    heads = list(sharding.shard_heads(41, rank, world))
    local_ms = 10.0 + 5.0 * rank                        # rank 1 is the slow one
    value, ms = sharding.aggregate_throughput(1000.0, local_ms, world)
    q.put((rank, heads, value, ms))
    dist.destroy_process_group()


def test_two_rank_sharding_and_max_over_ranks_timing():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    (r0, h0, v0, ms0), (r1, h1, v1, ms1) = res
    assert h0 == list(range(0, 21)) and h1 == list(range(21, 41))        # balanced, disjoint, complete
    assert ms0 == ms1 == 15.0                                            # max over ranks on both ranks
    assert v0 == v1 == 2 * 1000.0 / 15e-3


def test_shard_heads_covers_everything():
    from paper_2607_24377_b200 import sharding
    for n in (1, 7, 40, 41):
        for w in (1, 2, 3, 8):
            got = [h for r in range(w) for h in sharding.shard_heads(n, r, w)]
            assert got == list(range(n))
