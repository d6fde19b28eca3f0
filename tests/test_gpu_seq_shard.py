"""The two stages of a sequence-sharded forward (key_pass, query_pass) on one GPU: the ranks' ranges are processed
one after the other, their partial states are added and their softmax keys concatenated in rank order (what the
all-reduce and the all-gather do), and the assembled output is compared with the float64 oracle on the whole layer."""
import numpy as np
import pytest

from oracle import hybrid_attention as O
from paper_2509_24899_b200 import seq_shard as SS
from paper_2509_24899_b200 import workloads as W
from _util import assert_parity, balanced_gain, from_cuda_bf16, oracle_eval, oracle_inputs, oracle_mask, to_cuda_bf16

pytestmark = pytest.mark.gpu

CASES = {
    "ragged_d128": W.Workload("ss_ragged_d128", B=1, H=2, d=128, F=128, grid=(3, 10, 13), block=(1, 6, 8), rate=4, seed=71),
    "batch_d64": W.Workload("ss_batch_d64", B=2, H=3, d=64, F=64, grid=(2, 9, 31), block=(1, 4, 4), rate=2, seed=72,
                            rms_norm_qk=False),
    "chunks": W.Workload("ss_chunks", B=1, H=1, d=128, F=128, grid=(8, 30, 52), block=(1, 6, 8), rate=8, seed=73),
    "paper_phi": W.Workload("ss_paper_phi", B=1, H=2, d=128, F=256, grid=(3, 10, 13), block=(1, 6, 8), rate=4, seed=74,
                            layers=2, hidden=256),
    "rate0": W.Workload("ss_rate0", B=1, H=2, d=128, F=128, grid=(3, 10, 13), block=(1, 6, 8), rate=0, seed=75),
    "rate1": W.Workload("ss_rate1", B=1, H=2, d=128, F=128, grid=(3, 10, 13), block=(1, 6, 8), rate=1, seed=76),
}


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("mode", [O.STAB_PAPER, O.STAB_EXACT])
@pytest.mark.parametrize("name", sorted(CASES))
def test_sharded_stages_reproduce_the_layer(name, mode, world):
    import torch
    from paper_2509_24899_b200 import HybridAttention
    wl = CASES[name]
    gain = balanced_gain(wl, mode)
    data = W.generate(wl, wq_gain=gain)
    dev = {k: to_cuda_bf16(v) for k, v in data.items()}
    mask = oracle_mask(wl)
    idx = np.flatnonzero(mask).tolist()
    ranges = SS.token_ranges(wl.N, world)
    kw = dict(phi_dim=wl.F, poly_degree=wl.degree, stab_mode=mode, phi_layers=wl.layers, phi_hidden=wl.hidden_width)
    wts = dict(wq2=dev.get("wq2"), wk2=dev.get("wk2"))
    ops, keys = [], []
    for n0, n1 in ranges:                                         # stage 1 on every range
        n = n1 - n0
        op = HybridAttention(wl.B, wl.H, n, wl.d, (1, 1, n), (1, 1, n), 2, softmax_idx=SS.local_softmax_indices(idx, n0, n1), **kw)
        k_loc, v_loc = dev["k"][:, :, n0:n1].contiguous(), dev["v"][:, :, n0:n1].contiguous()
        ks, vs, S, z = op.key_pass(k_loc, v_loc, dev["wq"], dev["wk"], **wts)
        keys.append((ks.clone(), vs.clone(), S.clone(), z.clone()))
        ops.append(op)
    any_linear = len(idx) < wl.N
    ks = torch.cat([t[0] for t in keys], dim=1).contiguous()       # the all-gather: rows in rank order
    vs = torch.cat([t[1] for t in keys], dim=1).contiguous()
    S = sum(t[2] for t in keys) if any_linear else None            # the all-reduce
    z = sum(t[3] for t in keys) if any_linear else None
    outs = []
    for (n0, n1), op in zip(ranges, ops):                          # stage 2 on every range
        q_loc = dev["q"][:, :, n0:n1].contiguous()
        outs.append(op.query_pass(q_loc, dev["wq"], dev["wk"], ks, vs, S, z, **wts))
    torch.cuda.synchronize()
    assert all(op.last_status() == 0 for op in ops)
    got = from_cuda_bf16(torch.cat(outs, dim=2))
    ref, _ = oracle_eval(wl, oracle_inputs(data), mode)
    ok = np.isfinite(ref).all(-1)
    assert ok.mean() > 0.99
    assert_parity(got[ok], ref[ok], "seq_shard/%s/world%d/%s" % (name, world, "exact" if mode == O.STAB_EXACT else "paper"))
