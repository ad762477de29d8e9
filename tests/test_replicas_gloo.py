"""The N > 1 path is replicas over token shards: host-side sharding and the max-over-ranks timing protocol, run as
two gloo ranks on CPU."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_19438_b200 import replicas


def test_token_shards_tile_the_batch():
    for m, w in [(2048, 8), (2049, 8), (5, 8), (0, 3), (100, 1)]:
        spans = [replicas.shard_tokens(m, w, r) for r in range(w)]
        assert spans[0][0] == 0 and sum(c for _, c in spans) == m
        for (s0, c0), (s1, _) in zip(spans, spans[1:]):
            assert s0 + c0 == s1
        assert max(c for _, c in spans) - min(c for _, c in spans) <= 1


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dist.barrier()
        mine = 1.0 + rank                       # rank 1 is the slow one
        worst = replicas.max_over_ranks(mine)
        start, cnt = replicas.shard_tokens(2049, world, rank)
        tot = torch.tensor([cnt], dtype=torch.int64)
        dist.all_reduce(tot)
        q.put((rank, worst, start, cnt, int(tot.item()), replicas.whole_job_rate(100.0, world, worst)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [2.0, 2.0]
    assert res[0][2:4] == (0, 1025) and res[1][2:4] == (1025, 1024)
    assert res[0][4] == 2049 and res[0][5] == 100.0
    assert replicas.max_over_ranks(3.5) == 3.5     # no process group: identity
