"""Row-sharded gossip round: the deployment the paper describes, with the workers of one job
spread over several GPUs (one process per GPU, `per_rank` consecutive workers each).

A matched pair whose two workers live on the same GPU is averaged in place by the fused
round.  A pair that straddles two GPUs really exchanges its packed buffer (Algorithm 2:
ExchangeModelWithPeer): the same fused pass that applies the SGD step also writes every
worker's packed buffer (saps_round_pack; a worker whose peer is remote is a single row of that
pass, so what it emits is its post-SGD model at the kept coordinates) -> one send and one
receive of `cap` floats per such worker (torch.distributed point-to-point, NCCL over NVLink on
GPUs) -> saps_unpack_avg_rows.  Received buffers land in this GPU's own memory before any kernel
reads them.  Buffers travel at their full capacity `cap` (a few percent more than `count`),
so no device-to-host read of the count is needed before sending.

`plan_row_exchange` is pure host logic; `exchange_rows` is the only communication step.

Direct form (`destination_table`, `RowShardedGossip.local_step_direct`): where the GPUs can store
into one another's memory (peer access over NVLink; the receive buffers mapped into every process,
e.g. through CUDA IPC handles or a symmetric-memory allocation), the fused pass writes each
remote-peer worker's packed values straight into the receiving rank's buffer
(saps_round_pack_rows) and no transfer step follows: only "my pass has finished" has to reach the
peer (stream synchronisation, then a barrier of the process group) before it merges.  That form
has run with both ranks' buffers on one GPU only.
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass(frozen=True)
class RowExchangePlan:
    local_pairs: tuple      # involution on this rank's local rows: intra-rank pairs, else self
    transfers: tuple        # (local_row, peer_rank, tag) for every local worker whose peer is remote
    src_rows: tuple         # per local row: the row of the receive buffer to average with, or -1


def plan_row_exchange(pairs, rank: int, world: int, per_rank: int) -> RowExchangePlan:
    """Split a global matching (involution on world * per_rank workers) into what this rank
    averages locally and what it has to exchange.  The tag of a transfer is the smaller global
    worker index of the pair, the same on both sides."""
    n = world * per_rank
    pairs = [int(v) for v in pairs]
    if len(pairs) != n or any(not (0 <= pairs[i] < n) or pairs[pairs[i]] != i for i in range(n)):
        raise ValueError("pairs is not an involution on world * per_rank workers")
    lo = rank * per_rank
    local_pairs, transfers, src_rows = [], [], []
    for r in range(per_rank):
        j = pairs[lo + r]
        if lo <= j < lo + per_rank:
            local_pairs.append(j - lo)
            src_rows.append(-1)
        else:
            local_pairs.append(r)
            transfers.append((r, j // per_rank, min(lo + r, j)))
            src_rows.append(r)
    return RowExchangePlan(tuple(local_pairs), tuple(transfers), tuple(src_rows))


def destination_table(plan: RowExchangePlan, pairs, rank: int, per_rank: int, recv_base_of_rank, cap: int):
    """Per local worker, the address its packed values should be written to (for
    saps_round_pack_rows): row j of rank q's receive buffer when its peer is local row j of rank q
    (recv_base_of_rank[q] is the address of that [per_rank, cap] fp32 buffer as THIS process sees
    it), 0 when the peer is local (nothing to send).  The receiver finds the buffer of the worker
    that local row j is paired with in row j, which is what plan.src_rows says."""
    table = [0] * per_rank
    for r, peer_rank, _tag in plan.transfers:
        j = int(pairs[rank * per_rank + r]) - peer_rank * per_rank
        table[r] = int(recv_base_of_rank[peer_rank]) + 4 * cap * j
    return table


def exchange_rows(send, recv, plan: RowExchangePlan, group=None) -> None:
    """send, recv: [per_rank, cap] tensors (device for NCCL, CPU for gloo).  For every transfer
    of the plan, row r of `send` goes to the peer rank and the peer's row arrives in row r of
    `recv`.  Returns when the received rows are usable."""
    import torch.distributed as dist
    if not plan.transfers:
        return
    ops = []
    # both sides order their transfers by tag, so the k-th send of one rank to another meets
    # the k-th receive there even when two ranks share several pairs
    for r, peer, _tag in sorted(plan.transfers, key=lambda tr: tr[2]):
        ops.append(dist.P2POp(dist.isend, send[r], peer, group))
        ops.append(dist.P2POp(dist.irecv, recv[r], peer, group))
    for req in dist.batch_isend_irecv(ops):
        req.wait()


class RowShardedGossip:
    """One rank's share of the workers and the per-round sequence of library calls."""

    def __init__(self, rank: int, world: int, per_rank: int, N: int, ld: int, seed: int):
        from . import binding as sb
        self.sb, self.rank, self.world, self.per_rank = sb, rank, world, per_rank
        self.ctx = sb.saps_create_ld(per_rank, N, ld, seed)

    def close(self):
        self.sb.saps_destroy(self.ctx)

    def local_step(self, x, g, lr, pairs, t, keep_frac, vals, idx, count):
        """SGD step for every local worker, average of the pairs that live here, and the packed
        buffers of the workers whose peer is remote.  Returns the exchange plan."""
        sb = self.sb
        plan = plan_row_exchange(pairs, self.rank, self.world, self.per_rank)
        if plan.transfers:
            # one pass: SGD step, local averages, and the wire buffers (values before any average)
            sb.saps_round_pack(self.ctx, x, g, lr, plan.local_pairs, t, keep_frac, vals, idx, count)
        else:
            sb.saps_round(self.ctx, x, g, lr, plan.local_pairs, t, keep_frac)
        return plan

    def local_step_direct(self, x, g, lr, pairs, t, keep_frac, recv_base_of_rank, table_dev, idx, count):
        """As local_step, but the packed values of the workers whose peer is remote are written by
        the fused pass itself into the peers' receive buffers.  table_dev: device int64 tensor of
        per_rank entries that this call fills (it must stay untouched until the pass has run)."""
        import torch
        sb = self.sb
        plan = plan_row_exchange(pairs, self.rank, self.world, self.per_rank)
        if plan.transfers:
            cap = sb.saps_pack_capacity(self.ctx, keep_frac)
            table = destination_table(plan, pairs, self.rank, self.per_rank, recv_base_of_rank, cap)
            table_dev.copy_(torch.tensor(table, dtype=torch.int64), non_blocking=False)
            sb.saps_round_pack_rows(self.ctx, x, g, lr, plan.local_pairs, t, keep_frac, table_dev, idx, count)
        else:
            sb.saps_round(self.ctx, x, g, lr, plan.local_pairs, t, keep_frac)
        return plan

    def merge(self, x, plan, recv, idx, count, keep_frac):
        """Average the kept coordinates of the workers that received a buffer."""
        if plan.transfers:
            self.sb.saps_unpack_avg_rows(self.ctx, x, recv, idx, count, keep_frac, plan.src_rows)

    def round(self, x, g, lr, pairs, t, keep_frac, vals, idx, count, recv, group=None):
        """x, g: this rank's [per_rank, ld] matrices; pairs: the GLOBAL matching; vals/recv:
        [per_rank, cap] device buffers, idx [cap], count [1]."""
        plan = self.local_step(x, g, lr, pairs, t, keep_frac, vals, idx, count)
        exchange_rows(vals, recv, plan, group)
        self.merge(x, plan, recv, idx, count, keep_frac)
        return plan
