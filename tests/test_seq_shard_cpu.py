"""Sequence sharding, host side, on CPU with gloo ranks (no GPU, no kernels).

The driver (`seq_shard.run_sharded`), the token ranges, the per-range index lists and the two collectives run as
they do on GPUs; the two stages are played by the float64 oracle, so that the assembled result can be compared
with the oracle on the whole layer: a wrong range, a wrong row order in the gather or a state that was not summed
shows as a wrong output."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from oracle import hybrid_attention as O                      # noqa: E402
from paper_2509_24899_b200 import seq_shard as SS              # noqa: E402


def _layer(N, R, seed):
    rng = np.random.default_rng(seed)
    H, d, F = 2, 4, 6
    q, k, v = (rng.standard_normal((1, H, N, d)) for _ in range(3))
    wq, wk = rng.uniform(-0.7, 0.7, (H, F, d)), rng.uniform(-0.7, 0.7, (H, F, d))
    mask = O.softmax_token_mask((1, 1, N), (1, 1, N), R)
    return q, k, v, wq, wk, mask


def _rank_output(rank, world, N, R, seed, mode):
    """What one rank computes: its stages are the oracle on its token range."""
    q, k, v, wq, wk, mask = _layer(N, R, seed)
    H, d, F = q.shape[1], q.shape[3], wq.shape[1]
    idx = np.flatnonzero(mask).tolist()
    ranges = SS.token_ranges(N, world)
    n0, n1 = ranges[rank]
    per_rank = [len(SS.local_softmax_indices(idx, a, b)) for a, b in ranges]
    loc = np.zeros(n1 - n0, bool)
    loc[SS.local_softmax_indices(idx, n0, n1)] = True

    def stage_keys():
        ks = torch.from_numpy(np.stack([k[0, h, n0:n1][loc] for h in range(H)]))
        vs = torch.from_numpy(np.stack([v[0, h, n0:n1][loc] for h in range(H)]))
        S, z = np.zeros((H, F, d)), np.zeros((H, F))
        if not loc.all():
            for h in range(H):
                S[h], z[h] = O.linear_state(k[0, h, n0:n1], v[0, h, n0:n1], wk[h], loc)
        return ks, vs, torch.from_numpy(S), torch.from_numpy(z)

    def stage_queries(ks, vs, S, z):
        # the hybrid equation for this range's queries, written out with the gathered keys and the summed state
        out = np.empty((H, n1 - n0, d))
        for h in range(H):
            qb = q[0, h, n0:n1]
            num, den = np.zeros((n1 - n0, d)), np.zeros(n1 - n0)
            lam = np.ones(n1 - n0)
            if ks.shape[1] > 0:
                s = qb @ ks[h].numpy().T / np.sqrt(d)
                c = s.max(1)
                e = np.exp(s - c[:, None])
                num, den = e @ vs[h].numpy(), e.sum(1)
                if mode == O.STAB_EXACT:
                    lam = np.exp(-c)
            if S is not None:
                fq = O.phi_features(qb, wq[h])
                num = num + lam[:, None] * (fq @ S[h].numpy())
                den = den + lam * (fq @ z[h].numpy())
            out[h] = num / den[:, None]
        return out

    return SS.run_sharded(stage_keys, stage_queries, SS.TorchComm(), per_rank, len(idx) < N), (n0, n1)


def _worker(rank, world, port, out_dir, N, R, seed, mode):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    out, (n0, n1) = _rank_output(rank, world, N, R, seed, mode)
    np.save(os.path.join(out_dir, "rank%d.npy" % rank), out)
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("N,R,mode,port", [(37, 3, O.STAB_PAPER, 29551), (40, 4, O.STAB_EXACT, 29552),
                                           (23, 1, O.STAB_PAPER, 29553), (23, 0, O.STAB_PAPER, 29554)])
def test_two_ranks_reproduce_the_unsharded_layer(tmp_path, N, R, mode, port):
    world, seed = 2, 7
    mp.spawn(_worker, args=(world, port, str(tmp_path), N, R, seed, mode), nprocs=world, join=True)
    got = np.concatenate([np.load(tmp_path / ("rank%d.npy" % r)) for r in range(world)], axis=1)   # rows in rank order
    q, k, v, wq, wk, mask = _layer(N, R, seed)
    ref, _ = O.hybrid_attention(q, k, v, wq, wk, mask, None, mode)
    np.testing.assert_allclose(got, ref[0], rtol=1e-10, atol=1e-12)


def test_ranges_and_index_lists():
    assert SS.token_ranges(10, 3) == [(0, 4), (4, 7), (7, 10)]
    assert SS.token_ranges(4, 4) == [(0, 1), (1, 2), (2, 3), (3, 4)]
    idx = [0, 3, 4, 9]
    parts = [SS.local_softmax_indices(idx, a, b) for a, b in SS.token_ranges(10, 3)]
    assert parts == [[0, 3], [0], [2]]
    # every softmax token belongs to exactly one range, and the ranges in order give the list back
    back = [i + a for (a, _), p in zip(SS.token_ranges(10, 3), parts) for i in p]
    assert back == idx
