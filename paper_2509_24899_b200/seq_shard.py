"""Sequence sharding of one hybrid-attention layer over the ranks of a torch.distributed group.

Every rank owns a contiguous range of the layer's tokens (its rows of q, k, v and of the output).  The linear
state S, z is a sum over keys that does not depend on the query, so the ranks' partial states add up (one
all-reduce of [B*H, F, d+1] floats), and the softmax tokens of the ranges, taken in rank order, are the layer's
softmax tokens in token order (one all-gather of the compacted K_S, V_S).  After these two exchanges every rank
runs the query stage on its own rows.  Everything gathered lands in this rank's own memory before a kernel
reads it.

This module is plumbing: ranges, index lists, the two collectives and the order of the stages.  The arithmetic
of the stages is the library's (`HybridAttention.key_pass` / `query_pass`); `run_sharded` takes the stages as
callables, so that the same driver can be exercised on CPU ranks with any implementation of the two stages.
"""
from __future__ import annotations


def token_ranges(n_tokens: int, world: int):
    """Contiguous, near-equal token ranges [(n0, n1)] per rank; the first n_tokens % world ranks get one more."""
    base, extra = divmod(n_tokens, world)
    out, n0 = [], 0
    for r in range(world):
        n1 = n0 + base + (1 if r < extra else 0)
        out.append((n0, n1))
        n0 = n1
    return out


def local_softmax_indices(global_idx, n0: int, n1: int):
    """The softmax tokens of the range [n0, n1), counted from n0 (global_idx: sorted token indices of the layer)."""
    return [i - n0 for i in global_idx if n0 <= i < n1]


class TorchComm:
    """The two exchanges over a torch.distributed process group (NCCL on GPUs, gloo on CPU ranks)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self.world = dist.get_world_size(group)

    def all_reduce_sum(self, t):
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM, group=self.group)
        return t

    def all_gather_rows(self, t, rows_per_rank):
        """t: [BH, rows_per_rank[rank], d] -> [BH, sum(rows_per_rank), d], the ranks' rows in rank order.  Ranks may
        hold different numbers of rows: every rank sends a tensor padded to the largest count."""
        import torch
        most = max(rows_per_rank)
        if most == 0:
            return t
        padded = torch.zeros((t.shape[0], most, t.shape[2]), dtype=t.dtype, device=t.device)
        padded[:, :t.shape[1]] = t
        parts = [torch.empty_like(padded) for _ in range(self.world)]
        self.dist.all_gather(parts, padded, group=self.group)
        return torch.cat([p[:, :n] for p, n in zip(parts, rows_per_rank)], dim=1).contiguous()


def run_sharded(stage_keys, stage_queries, comm, softmax_per_rank, any_linear: bool):
    """One sequence-sharded forward on this rank.

    stage_keys()                      -> (ks, vs, S, z): this range's softmax keys / values [BH, n, d] and partial
                                         state [BH, F, d], [BH, F] (S, z ignored when not any_linear)
    stage_queries(ks, vs, S, z)       -> this range's output rows, from the gathered keys and the summed state
                                         (S = z = None when no rank has linear tokens)
    comm                              -> all_reduce_sum(tensor), all_gather_rows(tensor, rows_per_rank)
    softmax_per_rank                  -> number of softmax tokens of every rank's range"""
    ks, vs, S, z = stage_keys()
    if any_linear:
        S, z = comm.all_reduce_sum(S), comm.all_reduce_sum(z)
    else:
        S = z = None
    ks = comm.all_gather_rows(ks, softmax_per_rank)
    vs = comm.all_gather_rows(vs, softmax_per_rank)
    return stage_queries(ks, vs, S, z)


class SeqShardedAttention:
    """This rank's part of a layer whose tokens are spread over `world` ranks (CUDA; collectives over `group`)."""

    def __init__(self, B, H, N, d, global_softmax_idx, rank, world, group=None, comm=None, **handle_kw):
        from . import HybridAttention
        self.ranges = token_ranges(N, world)
        self.n0, self.n1 = self.ranges[rank]
        self.softmax_per_rank = [len(local_softmax_indices(global_softmax_idx, a, b)) for a, b in self.ranges]
        self.any_linear = len(global_softmax_idx) < N
        local_idx = local_softmax_indices(global_softmax_idx, self.n0, self.n1)
        n_loc = self.n1 - self.n0
        # the range as a layer of its own: a 1 x 1 x n grid with an explicit softmax-token list
        self.op = HybridAttention(B, H, n_loc, d, (1, 1, n_loc), (1, 1, n_loc), 2, softmax_idx=local_idx, **handle_kw)
        self.shape = (B, H, n_loc, d)
        self.comm = comm if comm is not None else TorchComm(group)

    def forward(self, q, k, v, wq=None, wk=None, out=None, aux=None, **weights):
        """q, k, v: this range's rows [B, H, n_loc, d] (contiguous bf16 CUDA tensors).  Returns the range's output."""
        def stage_keys():
            return self.op.key_pass(k, v, wq, wk, **weights)

        def stage_queries(ks, vs, S, z):
            return self.op.query_pass(q, wq, wk, ks, vs, S, z, out=out, aux=aux, **weights)

        return run_sharded(stage_keys, stage_queries, self.comm, self.softmax_per_rank, self.any_linear)
