"""The N > 1 path on CPU: two gloo ranks exercise the host logic that bench.py --gpus N uses
(column shards, identical matchings on every rank without communication, global placement of
the packed buffers, max-over-ranks timing)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2002_09692_b200 import sharding, synth


def test_column_shard_covers_everything_once():
    for n_total in (1, 2047, 2048, 2049, 14_728_266, 124_439_808):
        for world in (1, 2, 3, 8):
            spans = [sharding.column_shard(n_total, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n_total
            for (b0, e0), (b1, e1) in zip(spans, spans[1:]):
                assert e0 == b1 and b0 <= e0
            for b, e in spans:
                assert b % sharding.TILE_COLS == 0 or b == n_total
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 2 * sharding.TILE_COLS
    with pytest.raises(ValueError):
        sharding.weak_shard(1 << 30, 8, 0)
    assert sharding.weak_shard(14_728_266, 8, 7) == (7 * 14_728_266, 14_728_266)
    assert sharding.exclusive_offsets([3, 0, 5]) == ([0, 3, 3], 8)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, n_total, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2002_09692_b200 import binding as sb
        n, seed, p, T = 8, 3, 0.05, 6
        begin, end = sharding.column_shard(n_total, world, rank)
        # every rank selects its peers on its own: same seed, t and bandwidth -> same matching
        B = synth.bandwidth_matrix(n, 1.0, 100.0, seed=seed)
        ctx = sb.saps_create(n, max(1, end - begin), seed)
        sb.saps_set_column_offset(ctx, begin)
        mine = [sb.saps_select_peers(ctx, B, t, n) for t in range(1, T + 1)]
        sb.saps_destroy(ctx)
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        assert all(g == gathered[0] for g in gathered), "ranks disagree on the matching"
        # this shard's part of the round mask and its place in the global wire buffer
        m = oracle.mask(seed, 1, p, n_total)[begin:end]
        offset, total = sharding.global_pack_offset(int(m.sum()))
        slowest = sharding.max_over_ranks(10.0 + rank)
        results[rank] = (begin, end, int(m.sum()), offset, total, slowest)
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo():
    world, n_total = 2, 5 * 2048 + 300
    ctx = mp.get_context("spawn")
    with ctx.Manager() as mgr:
        results = mgr.dict()
        port = _free_port()
        procs = [ctx.Process(target=_worker, args=(r, world, port, n_total, results)) for r in range(world)]
        for pr in procs:
            pr.start()
        for pr in procs:
            pr.join(120)
            assert pr.exitcode == 0
        res = [results[r] for r in range(world)]
    full = oracle.mask(3, 1, 0.05, n_total)
    assert res[0][0] == 0 and res[0][1] == res[1][0] and res[1][1] == n_total
    assert res[0][3] == 0 and res[1][3] == res[0][2]                    # exclusive scan of the counts
    assert res[0][4] == res[1][4] == int(full.sum()) == res[0][2] + res[1][2]
    assert res[0][5] == res[1][5] == 11.0                               # the slowest rank's time


# ---- row-sharded deployment: planning and the exchange step, on CPU ranks ---------------------

def test_plan_row_exchange_splits_a_matching():
    from paper_2002_09692_b200.row_sharded import plan_row_exchange
    pairs = [1, 0, 5, 6, 7, 2, 3, 4]                     # 8 workers, 2 ranks of 4
    p0 = plan_row_exchange(pairs, 0, 2, 4)
    p1 = plan_row_exchange(pairs, 1, 2, 4)
    assert p0.local_pairs == (1, 0, 2, 3) and p0.src_rows == (-1, -1, 2, 3)
    assert p0.transfers == ((2, 1, 2), (3, 1, 3))
    assert p1.local_pairs == (3, 1, 2, 0) and p1.src_rows == (-1, 1, 2, -1)
    assert p1.transfers == ((1, 0, 2), (2, 0, 3))        # same tags as on rank 0
    with pytest.raises(ValueError):
        plan_row_exchange([1, 2, 0, 3], 0, 2, 2)


def test_destination_table_sends_every_row_where_its_receiver_looks():
    # Direct form: rank r's pass writes worker i's packed row to an address in the peer rank's
    # receive buffer.  With every "address" a (rank, row) code, following the tables of all ranks
    # must put, in row j of rank q's buffer, exactly the worker that row j's plan says it
    # averages with (src_rows[j] == j), and nothing anywhere else.
    from paper_2002_09692_b200.row_sharded import destination_table, plan_row_exchange
    world, per_rank, cap = 3, 4, 10
    rng = np.random.default_rng(11)
    bases = [1_000_000 * (q + 1) for q in range(world)]              # fake, well separated addresses
    for _ in range(20):
        pairs = synth.random_perfect_matching(world * per_rank, rng)
        plans = [plan_row_exchange(pairs, r, world, per_rank) for r in range(world)]
        arrived = {}                                                    # (rank, row) -> sending worker
        for r in range(world):
            table = destination_table(plans[r], pairs, r, per_rank, bases, cap)
            assert len(table) == per_rank
            for i, addr in enumerate(table):
                me = r * per_rank + i
                if int(pairs[me]) // per_rank == r:
                    assert addr == 0                                    # local pair: nothing to send
                    continue
                q, off = divmod(addr, 1_000_000)
                q -= 1
                assert off % (4 * cap) == 0
                assert (q, off // (4 * cap)) not in arrived
                arrived[(q, off // (4 * cap))] = me
        for q in range(world):
            for j in range(per_rank):
                peer = int(pairs[q * per_rank + j])
                if peer // per_rank == q:
                    assert (q, j) not in arrived and plans[q].src_rows[j] == -1
                else:
                    assert arrived[(q, j)] == peer and plans[q].src_rows[j] == j


def _row_worker(rank, world, port, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2002_09692_b200.row_sharded import exchange_rows, plan_row_exchange
        per_rank, cap = 4, 6
        rng = np.random.default_rng(5)
        ok = True
        for _ in range(5):
            pairs = synth.random_perfect_matching(world * per_rank, rng)     # same stream on both ranks
            plan = plan_row_exchange(pairs, rank, world, per_rank)
            send = torch.arange(per_rank * cap, dtype=torch.float32).reshape(per_rank, cap) + 1000.0 * rank
            recv = torch.full((per_rank, cap), -1.0)
            exchange_rows(send, recv, plan)
            for r in range(per_rank):
                j = int(pairs[rank * per_rank + r])
                if j // per_rank == rank:
                    ok &= bool((recv[r] == -1.0).all())                      # nothing arrives for local pairs
                else:
                    want = torch.arange(cap, dtype=torch.float32) + (j % per_rank) * cap + 1000.0 * (j // per_rank)
                    ok &= bool((recv[r] == want).all())                      # the peer's row, whole
        results[rank] = ok
    finally:
        dist.destroy_process_group()


def test_row_exchange_two_ranks_gloo():
    world = 2
    ctx = mp.get_context("spawn")
    with ctx.Manager() as mgr:
        results = mgr.dict()
        port = _free_port()
        procs = [ctx.Process(target=_row_worker, args=(r, world, port, results)) for r in range(world)]
        for pr in procs:
            pr.start()
        for pr in procs:
            pr.join(120)
            assert pr.exitcode == 0
        assert results[0] is True and results[1] is True
