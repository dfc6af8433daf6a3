"""World-size-2 CPU test (gloo) of the multi-rank bookkeeping used by bench.py --gpus N."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2502_03805_b200.dist_util import max_over_ranks, rank_layer_ids, whole_job_throughput


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    slowest = max_over_ranks(local_ms)
    dist.barrier()
    out.put((rank, slowest, rank_layer_ids(rank, 4)))
    dist.destroy_process_group()


def test_two_ranks_take_the_max_time_and_own_disjoint_layers():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]
    assert res[0][2] == [0, 1, 2, 3] and res[1][2] == [4, 5, 6, 7]
    assert whole_job_throughput(1000, 2, 0.015) == 2000 / 0.015


def _gather_worker(rank, world, port, out):
    import torch
    from paper_2502_03805_b200.dist_util import all_gather_heads, shard_kv_heads
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g0, g1 = shard_kv_heads(8, world, rank)
    full = torch.arange(2 * 8 * 5, dtype=torch.float32).reshape(2, 8, 5)
    got = all_gather_heads(full[:, g0:g1].contiguous())
    out.put((rank, (g0, g1), bool(torch.equal(got, full))))
    dist.destroy_process_group()


def test_kv_head_shards_gather_back_in_head_order():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_gather_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, (0, 4), True), (1, (4, 8), True)]


def test_kv_head_shards_reject_uneven_splits():
    import pytest
    from paper_2502_03805_b200.dist_util import shard_kv_heads
    assert [shard_kv_heads(8, 4, r) for r in range(4)] == [(0, 2), (2, 4), (4, 6), (6, 8)]
    with pytest.raises(ValueError):
        shard_kv_heads(8, 3, 0)
    with pytest.raises(ValueError):
        shard_kv_heads(8, 2, 2)


def test_single_process_is_identity():
    assert max_over_ranks(3.5) == 3.5


def _shard_worker(rank, world, port, out):
    """One rank of the KV-head-sharded mode on the CPU: its heads' group attention scores go through the real
    all-gather, the allocation is repeated on the gathered scores, and the rank keeps its slice of the budgets."""
    import numpy as np
    import torch
    from oracle import criticalkv_oracle as oc
    from paper_2502_03805_b200.dist_util import all_gather_heads, local_budget_slice, shard_kv_heads
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    nb, Hkv, n, btotal = 3, 8, 257, 600
    a_full = np.random.default_rng(5).random((nb, Hkv, n)).astype(np.float32) ** 4      # same on every rank
    g0, g1 = shard_kv_heads(Hkv, world, rank)
    a_all = all_gather_heads(torch.from_numpy(a_full[:, g0:g1].copy()))                  # what the GPU path gathers
    budgets = torch.tensor(np.stack([oc.allocate_budgets(a_all[b].numpy(), "adaptive", btotal) for b in range(nb)]),
                           dtype=torch.int32)
    mine = local_budget_slice(budgets, Hkv, world, rank)
    out.put((rank, (g0, g1), bool(torch.equal(a_all, torch.from_numpy(a_full))), mine.tolist(), budgets.tolist()))
    dist.destroy_process_group()


def test_sharded_mode_gathers_scores_and_slices_budgets_consistently():
    import numpy as np
    from oracle import criticalkv_oracle as oc
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    world = 2
    procs = [ctx.Process(target=_shard_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    a_full = np.random.default_rng(5).random((3, 8, 257)).astype(np.float32) ** 4
    want = [oc.allocate_budgets(a_full[b], "adaptive", 600).tolist() for b in range(3)]
    for rank, (g0, g1), gathered_ok, mine, budgets in res:
        assert gathered_ok and (g0, g1) == (4 * rank, 4 * rank + 4)
        assert budgets == want                                   # every rank repeats the same allocation
        assert mine == [row[g0:g1] for row in want]              # and keeps the columns of its own heads
    assert all(sum(r0 + r1) == 600 for r0, r1 in zip(res[0][3], res[1][3]))
