"""Host-side logic of the multi-GPU (row-sharded) path, run as two gloo ranks on CPU."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_29860_b200 import shard


def test_shard_rows_is_a_partition():
    for n, w in ((512, 1), (512, 8), (513, 8), (7, 3), (3, 8), (0, 4)):
        parts = shard.shard_rows(n, w)
        assert len(parts) == w and parts[0][0] == 0 and parts[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
        sizes = [hi - lo for lo, hi in parts]
        assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard.shard_rows(4, 0)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    plan = shard.rank_plan(rank, world, rows_per_rank=512)
    ms = shard.max_over_ranks([10.0 + rank, 5.0 - rank], dist)           # per-rank timings -> max over ranks
    tot = shard.sum_over_ranks([512.0, float(rank)], dist)
    seeds = [None] * world
    dist.all_gather_object(seeds, (plan["state_seed"], plan["data_seed_offset"], plan["rows"]))
    # vocabulary shards: each rank contributes its partials, everyone ends with [world, rows, 8] in rank order
    mine = torch.full((5, 8), float(rank + 1)) + torch.arange(5, dtype=torch.float32)[:, None]
    gathered = shard.all_gather_partials(mine, dist)
    stats = shard.all_gather_batch_stats([1.0 + rank, 0.5, 0.25, 100 * (rank + 1), 10, 2 + rank], dist)
    torch.save({"ms": ms, "tot": tot, "seeds": seeds, "plan": plan, "gathered": gathered, "stats": stats}, os.path.join(out_dir, f"r{rank}.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_rows_and_reduce_timings(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [torch.load(os.path.join(tmp_path, f"r{r}.pt")) for r in range(world)]
    for r in res:
        assert r["ms"] == [11.0, 5.0]                    # max over ranks, element-wise, same on every rank
        assert r["tot"] == [1024.0, 1.0]
        assert r["plan"]["global_rows"] == 1024
        assert r["stats"] == [[1.0, 0.5, 0.25, 100.0, 10.0, 2.0], [2.0, 0.5, 0.25, 200.0, 10.0, 3.0]]
        g = r["gathered"]
        assert tuple(g.shape) == (world, 5, 8) and g.is_contiguous()
        for k in range(world):
            assert torch.equal(g[k], torch.full((5, 8), float(k + 1)) + torch.arange(5, dtype=torch.float32)[:, None])
    seeds = res[0]["seeds"]
    assert len({s[0] for s in seeds}) == world and len({s[1] for s in seeds}) == world   # no shared noise or data
    assert [s[2] for s in seeds] == [(0, 512), (512, 1024)]                               # disjoint, contiguous rows


def test_vocab_shards_cover_the_vocabulary():
    for V, w in ((152064, 8), (152064, 1), (128256, 4), (32000, 3), (1000, 8), (5, 2)):
        parts = shard.vocab_shards(V, w)
        assert len(parts) == w and parts[0][0] == 0 and sum(n for _, n in parts) == V
        assert all(lo % 128 == 0 or n == 0 for lo, n in parts)
        assert all(a[0] + a[1] == b[0] for a, b in zip(parts, parts[1:]))
    assert shard.all_gather_partials(torch.zeros(3, 8)).shape == (1, 3, 8)      # no process group: one shard
    with pytest.raises(ValueError):
        shard.vocab_shards(100, 2, multiple=6)
