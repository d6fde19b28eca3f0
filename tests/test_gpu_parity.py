"""Parity of the CUDA library (through the C ABI) against the float64 oracle.

Bar: relative L2 <= 5e-3 and max-abs <= 2e-2 x RMS(oracle output) for the bf16 output;
bit-exact for the integer token split.  Small cases are compared element by element; the
full-size configurations are compared on sampled query rows (every key still takes part in
each sampled row) plus the complete linear state S, z.
"""
import dataclasses
import math

import numpy as np
import pytest

from oracle import hybrid_attention as O
from paper_2509_24899_b200 import workloads as W
from _util import (Guarded, assert_parity, balanced_gain, errors, from_cuda_bf16, oracle_eval, oracle_inputs,
                   oracle_mask, oracle_state, to_cuda_bf16)

pytestmark = pytest.mark.gpu

PATHS = ["simt", "tensor"]
FULL_PATH = "tensor"          # path used at the full benchmark sizes
MODES = [O.STAB_PAPER, O.STAB_EXACT]

# ragged cases: N and N_S are not multiples of the 128-token tile
SMALL = {
    "ragged_d128": W.Workload("ragged_d128", B=1, H=2, d=128, F=128, grid=(3, 10, 13), block=(1, 6, 8),
                              rate=4, seed=11),
    "ragged_d64": W.Workload("ragged_d64", B=2, H=3, d=64, F=64, grid=(2, 9, 31), block=(1, 4, 4),
                             rate=2, seed=12, rms_norm_qk=False),
    "one_tile": W.Workload("one_tile", B=1, H=1, d=128, F=128, grid=(1, 5, 7), block=(1, 5, 7),
                           rate=3, seed=13),
    "paper_rule_1d": W.Workload("paper_rule_1d", B=1, H=2, d=128, F=128, grid=(1, 1, 1000),
                                block=(1, 1, 1000), rate=8, seed=14),
    "multi_chunk": W.Workload("multi_chunk", B=1, H=1, d=128, F=128, grid=(8, 30, 52), block=(1, 6, 8),
                              rate=8, seed=15),
}


def _path(name):
    from paper_2509_24899_b200 import AS_PATH_SIMT, AS_PATH_TENSOR
    return {"simt": AS_PATH_SIMT, "tensor": AS_PATH_TENSOR}[name]


def _run(wl, path, mode, gain=1.0, rows=None, heads=None, want_state=False, softmax_idx=None):
    """Runs the library on wl's inputs; returns (gpu out, gpu aux, oracle y, oracle aux, extras).

    out, aux and the workspace sit between sentinel-filled guard bands that must come back untouched."""
    import torch
    from paper_2509_24899_b200 import HybridAttention
    data = W.generate(wl, wq_gain=gain, heads=heads)
    if heads is not None:
        wl = dataclasses.replace(wl, H=heads)
    dev = {k: to_cuda_bf16(v) for k, v in data.items()}
    op = HybridAttention.from_workload(wl, stab_mode=mode, kernel_path=_path(path), softmax_idx=softmax_idx)
    n_el = wl.B * wl.H * wl.N
    g_out, g_aux, g_ws = Guarded(n_el * wl.d * 2), Guarded(n_el * 3 * 4), Guarded(op.workspace_bytes)
    out = g_out.view(torch.bfloat16, (wl.B, wl.H, wl.N, wl.d))
    aux = g_aux.view(torch.float32, (wl.B, wl.H, wl.N, 3))
    aux.fill_(float("nan"))
    op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"], out=out, aux=aux, workspace=g_ws.bytes(),
               wq2=dev.get("wq2"), wk2=dev.get("wk2"), biases={n: t for n, t in dev.items() if n.startswith("b")} or None)
    torch.cuda.synchronize()
    assert op.last_status() == 0
    for g, name in ((g_out, "out"), (g_aux, "aux"), (g_ws, "workspace")):
        g.check("%s/%s %s" % (wl.name, path, name))
    got = from_cuda_bf16(out)
    got_aux = aux.cpu().numpy().astype(np.float64)
    extras = {"op": op, "n_softmax": op.n_softmax, "indices": op.softmax_indices()}
    if want_state and op.n_softmax < wl.N:
        S, z = op.linear_state()
        torch.cuda.synchronize()
        extras["S"], extras["z"] = S.cpu().numpy().astype(np.float64), z.cpu().numpy().astype(np.float64)
    d64 = oracle_inputs(data)
    key = (wl, mode, float(gain), None if rows is None else tuple(int(r) for r in rows),
           None if softmax_idx is None else tuple(softmax_idx))
    ref, ref_aux = oracle_eval(wl, d64, mode, rows=rows, key=key)
    if rows is not None:
        got, got_aux = got[:, :, rows], got_aux[:, :, rows]
    extras["data64"] = d64
    extras["wl"] = wl
    return got, got_aux, ref, ref_aux, extras


def _tag(name, path, mode, balanced=None):
    t = "%s/%s/%s" % (name, path, "exact" if mode == O.STAB_EXACT else "paper")
    return t if balanced is None else t + ("/balanced" if balanced else "/as-drawn")


def _check_aux(got_aux, ref_aux, wl, n_softmax):
    if n_softmax > 0:
        np.testing.assert_allclose(got_aux[..., 0], ref_aux[..., 0], atol=2e-3, rtol=0)
        assert errors(got_aux[..., 1], ref_aux[..., 1])[0] <= 5e-3
    if n_softmax < wl.N:
        assert errors(got_aux[..., 2], ref_aux[..., 2])[0] <= 5e-3


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("balanced", [False, True])
def test_tiny_config(path, mode, balanced):
    wl = W.CONFIGS["tiny"]
    gain = balanced_gain(wl, mode) if balanced else 1.0
    got, got_aux, ref, ref_aux, ex = _run(wl, path, mode, gain, want_state=True)
    assert ex["n_softmax"] == 32
    assert_parity(got, ref, _tag("tiny", path, mode, balanced))
    _check_aux(got_aux, ref_aux, wl, 32)
    S, z = oracle_state(wl, ex["data64"])
    assert errors(ex["S"], S)[0] <= 5e-3 and errors(ex["z"], z)[0] <= 5e-3
    if balanced:
        lam = np.exp(-ref_aux[..., 0]) if mode == O.STAB_EXACT else 1.0
        ratio = np.median(lam * ref_aux[..., 2] / ref_aux[..., 1])
        assert 0.2 < ratio < 5.0          # both branches carry weight in this variant


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("name", sorted(SMALL))
def test_small_ragged_cases(path, mode, name):
    wl = SMALL[name]
    gain = balanced_gain(wl, mode)
    got, got_aux, ref, ref_aux, ex = _run(wl, path, mode, gain, want_state=True)
    mask = oracle_mask(wl)
    assert ex["indices"] == np.flatnonzero(mask).tolist()         # integer work: bit-exact
    assert_parity(got, ref, _tag(name, path, mode, True))
    _check_aux(got_aux, ref_aux, wl, int(mask.sum()))
    S, z = oracle_state(wl, ex["data64"])
    assert errors(ex["S"], S)[0] <= 5e-3 and errors(ex["z"], z)[0] <= 5e-3


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("rate", [0, 1])
@pytest.mark.parametrize("name", ["ragged_d128", "ragged_d64"])
def test_degenerate_rates(path, rate, name):
    wl = SMALL[name].with_rate(rate)
    got, got_aux, ref, ref_aux, ex = _run(wl, path, O.STAB_PAPER, want_state=(rate == 0))
    assert ex["n_softmax"] == (wl.N if rate == 1 else 0)
    ok = np.isfinite(ref).all(-1)          # rate 0: a query with all-zero features is NaN in both
    assert ok.mean() > 0.99
    assert_parity(got[ok], ref[ok], _tag("%s/R%d" % (name, rate), path, O.STAB_PAPER))
    _check_aux(got_aux[ok], ref_aux[ok], wl, ex["n_softmax"])
    if rate == 1:
        # rate 1 is plain softmax attention: cross-check with the library routine as well
        import torch
        d = ex["data64"]
        sd = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(d["q"]), torch.from_numpy(d["k"]), torch.from_numpy(d["v"])).numpy()
        assert_parity(got, sd, _tag("%s/R1-vs-sdpa" % name, path, O.STAB_PAPER))


@pytest.mark.parametrize("path", PATHS)
def test_explicit_softmax_index_list(path):
    wl = SMALL["ragged_d128"]
    rng = np.random.default_rng(5)
    idx = np.sort(rng.choice(wl.N, size=77, replace=False))
    import torch
    from paper_2509_24899_b200 import HybridAttention
    data = W.generate(wl, wq_gain=2e-3)
    dev = {k: to_cuda_bf16(v) for k, v in data.items()}
    op = HybridAttention.from_workload(wl, kernel_path=_path(path), softmax_idx=idx.tolist())
    out = op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"])
    torch.cuda.synchronize()
    assert op.softmax_indices() == idx.tolist()
    d64 = oracle_inputs(data)
    mask = np.zeros(wl.N, bool)
    mask[idx] = True
    ref, _ = O.hybrid_attention(d64["q"], d64["k"], d64["v"], d64["wq"], d64["wk"], mask)
    assert_parity(from_cuda_bf16(out), ref, _tag("explicit_idx", path, O.STAB_PAPER))


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("mode", MODES)
def test_late_dominant_keys_move_the_reference_maximum(path, mode):
    """Softmax keys late in the sequence are scaled up so that the row maximum grows by far more than 2^8
    after the first key tiles: the kernels have to rescale their running sums on the way."""
    import torch
    from paper_2509_24899_b200 import HybridAttention
    wl = SMALL["multi_chunk"]                       # N = 12480, 1560 softmax tokens = 13 key tiles
    data = W.generate(wl, wq_gain=balanced_gain(wl, mode))
    mask = oracle_mask(wl)
    idx = np.flatnonzero(mask)
    k32 = W.bf16_bits_to_f32(data["k"]).copy()
    k32[:, :, idx[700:703]] *= 6.0                  # tile 5: scores up to ~6x the usual maximum
    k32[:, :, idx[1500:1502]] *= 12.0               # last tile: larger again
    data["k"] = W.f32_to_bf16_bits(k32)
    dev = {k: to_cuda_bf16(v) for k, v in data.items()}
    op = HybridAttention.from_workload(wl, stab_mode=mode, kernel_path=_path(path))
    aux = torch.full((wl.B, wl.H, wl.N, 3), float("nan"), dtype=torch.float32, device="cuda")
    out = op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"], aux=aux)
    torch.cuda.synchronize()
    assert op.last_status() == 0
    d64 = oracle_inputs(data)
    rows = _sample_rows(wl.N, 512, 7)
    ref, ref_aux = oracle_eval(wl, d64, mode, rows=rows)
    assert (ref_aux[..., 0] > 12.0).mean() > 0.2   # the scaled keys do dominate many rows (c_i far above the usual ~4)
    assert_parity(from_cuda_bf16(out)[:, :, rows], ref, _tag("late_dominant_keys", path, mode, True))
    _check_aux(aux.cpu().numpy().astype(np.float64)[:, :, rows], ref_aux, wl, int(mask.sum()))


@pytest.mark.parametrize("path", PATHS)
def test_key_permutation_within_sets_leaves_output_unchanged(path):
    """Property that holds at any size: permuting keys inside T_S and inside T_L changes nothing."""
    import torch
    from paper_2509_24899_b200 import HybridAttention
    wl = SMALL["ragged_d128"]
    data = W.generate(wl, wq_gain=balanced_gain(wl, O.STAB_PAPER))
    mask = oracle_mask(wl)
    rng = np.random.default_rng(9)
    perm = np.arange(wl.N)
    for sel in (mask, ~mask):
        ids = np.flatnonzero(sel)
        perm[ids] = rng.permutation(ids)
    dev = {k: to_cuda_bf16(v) for k, v in data.items()}
    op = HybridAttention.from_workload(wl, kernel_path=_path(path))
    a = from_cuda_bf16(op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"]))
    kp = to_cuda_bf16(np.ascontiguousarray(data["k"][:, :, perm]))
    vp = to_cuda_bf16(np.ascontiguousarray(data["v"][:, :, perm]))
    b = from_cuda_bf16(op.forward(dev["q"], kp, vp, dev["wq"], dev["wk"]))
    torch.cuda.synchronize()
    assert errors(b, a)[0] <= 5e-3


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("balanced", [False, True])
def test_wan17_full(path, mode, balanced):
    wl = W.CONFIGS["wan17"]
    gain = balanced_gain(wl, mode) if balanced else 1.0
    got, got_aux, ref, ref_aux, ex = _run(wl, path, mode, gain, want_state=True)
    assert ex["n_softmax"] == 975
    assert_parity(got, ref, _tag("wan17", path, mode, balanced))
    _check_aux(got_aux, ref_aux, wl, 975)
    S, z = oracle_state(wl, ex["data64"])
    assert errors(ex["S"], S)[0] <= 5e-3 and errors(ex["z"], z)[0] <= 5e-3


def _sample_rows(N, n, seed):
    rng = np.random.default_rng(seed)
    rows = rng.choice(N, size=n - 4, replace=False)
    return np.unique(np.concatenate([rows, [0, 1, N - 2, N - 1]]))      # include first / last tile rows


@pytest.mark.parametrize("path", PATHS)          # outermost: varies fastest, so both paths share one oracle run
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("balanced", [False, True])
def test_wan81_headline_sampled_rows(path, mode, balanced):
    """Headline shape in the launch configuration the benchmark times (tensor path), and on the fp32 check path."""
    wl = W.CONFIGS["wan81"]
    gain = balanced_gain(wl, mode) if balanced else 1.0
    rows = _sample_rows(wl.N, 160, 1)
    got, got_aux, ref, ref_aux, ex = _run(wl, path, mode, gain, rows=rows, want_state=True)
    assert ex["n_softmax"] == 4095
    assert ex["indices"] == np.flatnonzero(oracle_mask(wl)).tolist()
    assert_parity(got, ref, _tag("wan81/160rows", path, mode, balanced))
    _check_aux(got_aux, ref_aux, wl, 4095)
    S, z = oracle_state(wl, ex["data64"])
    assert errors(ex["S"], S)[0] <= 5e-3 and errors(ex["z"], z)[0] <= 5e-3


# (rate, mode, balanced): at rates 1 and 0 there is one branch only, so the mode and the gain change nothing
STACK_CASES = [(1, O.STAB_PAPER, False), (0, O.STAB_PAPER, False)] + \
              [(r, m, b) for r in (4, 16) for m in MODES for b in (False, True)]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("rate,mode,balanced", STACK_CASES)
def test_stack_layer_rates_sampled_rows(path, rate, mode, balanced):
    """One layer of each distinct rate of the 30-layer block-rate stack (rate 8 is the headline), all heads."""
    sched = W.stack_schedule(0)
    layer = sched.index(rate)
    wl = W.stack_layer(layer)
    assert wl.rate == rate
    gain = balanced_gain(wl, mode) if balanced else 1.0
    rows = _sample_rows(wl.N, 96, 2)
    got, got_aux, ref, ref_aux, ex = _run(wl, path, mode, gain, rows=rows, want_state=(rate != 1))
    assert ex["n_softmax"] == {1: 32760, 4: 8190, 16: 2100, 0: 0}[rate]
    ok = np.isfinite(ref).all(-1)
    assert ok.mean() > 0.99
    assert_parity(got[ok], ref[ok], _tag("stack/R%d/96rows" % rate, path, mode, balanced))
    _check_aux(got_aux[ok], ref_aux[ok], ex["wl"], ex["n_softmax"])
    if rate != 1:
        S, z = oracle_state(ex["wl"], ex["data64"])
        assert errors(ex["S"], S)[0] <= 5e-3 and errors(ex["z"], z)[0] <= 5e-3


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("balanced", [False, True])
def test_wan161_cfg_batch_sampled_rows(path, mode, balanced):
    wl = W.CONFIGS["wan161cfg"]
    gain = balanced_gain(wl, mode) if balanced else 1.0
    rows = _sample_rows(wl.N, 64, 3)
    got, got_aux, ref, ref_aux, ex = _run(wl, path, mode, gain, rows=rows)
    assert ex["n_softmax"] == 4100
    assert_parity(got, ref, _tag("wan161cfg/64rows", path, mode, balanced))
    _check_aux(got_aux, ref_aux, wl, 4100)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name", ["wan81", "wan161cfg"])
def test_whole_output_at_full_size(path, name):
    """Every output element of the headline layer and of the long CFG-batch layer against the oracle
    (balanced feature maps, so that both branches carry weight): a mis-addressed unit, half-unit or
    head of the persistent schedule cannot hide between sampled rows."""
    wl = W.CONFIGS[name]
    gain = balanced_gain(wl, O.STAB_PAPER)
    got, got_aux, ref, ref_aux, ex = _run(wl, path, O.STAB_PAPER, gain)
    assert_parity(got, ref, _tag(name + "/whole", path, O.STAB_PAPER, True))
    _check_aux(got_aux, ref_aux, wl, ex["n_softmax"])
    # per (batch, head) as well: one wrong head would be diluted 12- or 24-fold in the global figure
    for b in range(wl.B):
        for h in range(wl.H):
            assert errors(got[b, h], ref[b, h])[0] <= 5e-3, (b, h)


@pytest.mark.parametrize("path", PATHS)
def test_host_buffer_entry_point_matches_device_entry_point(path):
    import torch
    from paper_2509_24899_b200 import HybridAttention
    wl = SMALL["ragged_d64"]
    data = W.generate(wl, wq_gain=balanced_gain(wl, O.STAB_PAPER))
    dev = {k: to_cuda_bf16(v) for k, v in data.items()}
    op = HybridAttention.from_workload(wl, kernel_path=_path(path))
    ref = op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"]).clone()
    host = {k: torch.from_numpy(data[k].view(np.int16)).pin_memory() for k in ("q", "k", "v")}
    out_host = torch.empty_like(host["q"]).pin_memory()
    op.forward_host(host["q"], host["k"], host["v"], dev["wq"], dev["wk"], out_host)
    torch.cuda.synchronize()
    assert torch.equal(out_host, ref.view(torch.int16).cpu())


def test_run_to_run_determinism_and_launch_count():
    import torch
    from paper_2509_24899_b200 import HybridAttention, binding
    wl = SMALL["multi_chunk"]
    data = W.generate(wl, wq_gain=1e-3)
    dev = {k: to_cuda_bf16(v) for k, v in data.items()}
    op = HybridAttention.from_workload(wl, kernel_path=_path(FULL_PATH))
    a = op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"]).clone()
    b = op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"]).clone()
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    # K pass (its CTAs add the chunks' partial states up themselves: no launch of its own) and Q pass; twice
    assert binding.as_hybrid_attn_launch_count(op.handle) == 4
    binding.as_hybrid_attn_profile_enable(op.handle, True)
    op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"])
    ms, cnt = binding.as_hybrid_attn_profile_read(op.handle)
    assert cnt == [1, 0, 1] and ms[0] > 0 and ms[2] > 0


def test_expired_device_wait_is_reported_once_and_the_handle_recovers():
    """The time-out path in its safe form: a dedicated kernel's bounded wait runs out (nothing else is in flight),
    the status word is set, forwards on the handle do nothing until the word has been read, last_status reports
    the time-out once, and the next forward is correct again."""
    import torch
    from paper_2509_24899_b200 import HybridAttention, binding
    wl = SMALL["one_tile"]
    data = W.generate(wl, wq_gain=0.02)
    dev = {k: to_cuda_bf16(v) for k, v in data.items()}
    op = HybridAttention.from_workload(wl)
    good = op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"]).clone()
    torch.cuda.synchronize()
    assert op.last_status() == 0
    st = torch.cuda.current_stream().cuda_stream
    binding.as_hybrid_attn_debug_expire_wait(op.handle, 2_000_000, st)       # about a millisecond
    sentinel = torch.full_like(good, 7.0)
    op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"], out=sentinel)   # inert: kernels return at once
    torch.cuda.synchronize()
    assert torch.equal(sentinel, torch.full_like(good, 7.0))
    assert op.last_status() == binding.AS_ERR_DEVICE_TIMEOUT
    assert op.last_status() == 0                                               # read and cleared
    again = op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"])
    torch.cuda.synchronize()
    assert op.last_status() == 0 and torch.equal(again, good)


def test_gpu_argument_errors():
    import torch
    from paper_2509_24899_b200 import HybridAttention, binding, AsError
    wl = SMALL["one_tile"]
    op = HybridAttention.from_workload(wl)
    data = {k: to_cuda_bf16(v) for k, v in W.generate(wl).items()}
    out = torch.empty_like(data["q"])
    ws = op.workspace()
    with pytest.raises(AsError) as e:
        binding.as_hybrid_attn_forward(op.handle, data["q"].data_ptr(), data["k"].data_ptr(), data["v"].data_ptr(),
                                       data["wq"].data_ptr(), data["wk"].data_ptr(), out.data_ptr(), 0,
                                       ws.data_ptr(), op.workspace_bytes - 1, 0)
    assert e.value.status == binding.AS_ERR_WORKSPACE
    with pytest.raises(AsError) as e:
        binding.as_hybrid_attn_forward(op.handle, data["q"].data_ptr() + 2, data["k"].data_ptr(), data["v"].data_ptr(),
                                       data["wq"].data_ptr(), data["wk"].data_ptr(), out.data_ptr(), 0,
                                       ws.data_ptr(), op.workspace_bytes, 0)
    assert e.value.status == binding.AS_ERR_INVALID_ARG
    with pytest.raises(AsError) as e:      # linear tokens exist, so the feature-map weights are required
        binding.as_hybrid_attn_forward(op.handle, data["q"].data_ptr(), data["k"].data_ptr(), data["v"].data_ptr(),
                                       0, 0, out.data_ptr(), 0, ws.data_ptr(), op.workspace_bytes, 0)
    assert e.value.status == binding.AS_ERR_INVALID_ARG


TWO_LAYER = {
    "two_layer_d128": W.Workload("two_layer_d128", B=1, H=2, d=128, F=128, grid=(3, 10, 13), block=(1, 6, 8),
                                 rate=4, seed=31, layers=2),
    "two_layer_d64": W.Workload("two_layer_d64", B=2, H=3, d=64, F=64, grid=(2, 9, 31), block=(1, 4, 4),
                                rate=2, seed=32, rms_norm_qk=False, layers=2),
    "two_layer_rate0": W.Workload("two_layer_rate0", B=1, H=2, d=128, F=128, grid=(3, 10, 13), block=(1, 6, 8),
                                  rate=0, seed=33, layers=2),
    "two_layer_chunks": W.Workload("two_layer_chunks", B=1, H=1, d=128, F=128, grid=(8, 30, 52), block=(1, 6, 8),
                                   rate=8, seed=34, layers=2),
    # more (batch, head) pairs than SMs: several units per persistent CTA, with the weight tiles of the tail and the
    # last V tile competing for the three ring slots at every unit's end
    "two_layer_many_units": W.Workload("two_layer_many_units", B=2, H=80, d=128, F=128, grid=(1, 10, 30), block=(1, 5, 6),
                                       rate=3, seed=35, layers=2),
    "two_layer_many_units_rate0": W.Workload("two_layer_many_units_rate0", B=2, H=80, d=64, F=64, grid=(1, 10, 30),
                                             block=(1, 5, 6), rate=0, seed=36, layers=2, rms_norm_qk=False),
}

# Feature maps wider than the head ("Characterization of phi": d -> P*d -> P*d, Table of phi sizes), polynomial
# degrees up to 4, biases.  paper_default is the paper's default map: two layers, hidden = F = 2d, degree 2.
WIDE = {
    "f256_one_layer": W.Workload("f256_one_layer", B=1, H=2, d=128, F=256, grid=(3, 10, 13), block=(1, 6, 8), rate=4, seed=41),
    "f384_degree3": W.Workload("f384_degree3", B=1, H=2, d=128, F=384, grid=(3, 10, 13), block=(1, 6, 8), rate=4, seed=42, degree=3),
    "f512_degree4_bias": W.Workload("f512_degree4_bias", B=1, H=2, d=128, F=512, grid=(3, 10, 13), block=(1, 6, 8), rate=3,
                                    seed=43, degree=4, bias=True),
    "f128_degree4": W.Workload("f128_degree4", B=1, H=2, d=128, F=128, grid=(3, 10, 13), block=(1, 6, 8), rate=4, seed=44, degree=4),
    "f128_bias": W.Workload("f128_bias", B=1, H=2, d=128, F=128, grid=(3, 10, 13), block=(1, 6, 8), rate=4, seed=45, bias=True),
    "d64_f128": W.Workload("d64_f128", B=2, H=3, d=64, F=128, grid=(2, 9, 31), block=(1, 4, 4), rate=2, seed=46, rms_norm_qk=False),
    "d64_f256_bias": W.Workload("d64_f256_bias", B=1, H=2, d=64, F=256, grid=(2, 9, 31), block=(1, 4, 4), rate=2, seed=47,
                                rms_norm_qk=False, bias=True),
    "f256_rate0": W.Workload("f256_rate0", B=1, H=2, d=128, F=256, grid=(3, 10, 13), block=(1, 6, 8), rate=0, seed=48),
    "f256_many_units": W.Workload("f256_many_units", B=2, H=80, d=128, F=256, grid=(1, 10, 30), block=(1, 5, 6), rate=3, seed=49),
    "f256_chunks": W.Workload("f256_chunks", B=1, H=1, d=128, F=256, grid=(8, 30, 52), block=(1, 6, 8), rate=8, seed=50),
    "paper_default": W.Workload("paper_default", B=1, H=2, d=128, F=256, grid=(3, 10, 13), block=(1, 6, 8), rate=4, seed=51,
                                layers=2, hidden=256),
    "paper_default_bias": W.Workload("paper_default_bias", B=1, H=2, d=128, F=256, grid=(3, 10, 13), block=(1, 6, 8), rate=4,
                                     seed=52, layers=2, hidden=256, bias=True),
    "paper_default_rate0": W.Workload("paper_default_rate0", B=1, H=2, d=128, F=256, grid=(3, 10, 13), block=(1, 6, 8), rate=0,
                                      seed=53, layers=2, hidden=256),
    "paper_default_many_units": W.Workload("paper_default_many_units", B=2, H=80, d=128, F=256, grid=(1, 10, 30), block=(1, 5, 6),
                                           rate=3, seed=54, layers=2, hidden=256),
    "paper_default_chunks": W.Workload("paper_default_chunks", B=1, H=1, d=128, F=256, grid=(8, 30, 52), block=(1, 6, 8), rate=8,
                                       seed=55, layers=2, hidden=256),
    "hidden256_f128": W.Workload("hidden256_f128", B=1, H=2, d=128, F=128, grid=(3, 10, 13), block=(1, 6, 8), rate=4, seed=56,
                                 layers=2, hidden=256),
    "hidden128_f256_bias": W.Workload("hidden128_f256_bias", B=1, H=2, d=128, F=256, grid=(3, 10, 13), block=(1, 6, 8), rate=4,
                                      seed=57, layers=2, hidden=128, bias=True),
    "two_layer_d64_bias": W.Workload("two_layer_d64_bias", B=2, H=3, d=64, F=64, grid=(2, 9, 31), block=(1, 4, 4), rate=2, seed=58,
                                     rms_norm_qk=False, layers=2, bias=True),
}
FEATURE_MAPS = dict(TWO_LAYER, **WIDE)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("name", sorted(FEATURE_MAPS))
def test_feature_map_shapes(mode, name):
    """Deeper and wider feature maps: two layers (first layer of the keys by its own kernel, of the queries inside the
    Q pass), up to 512 features in chunks of 128, polynomial degrees up to 4, biases."""
    wl = FEATURE_MAPS[name]
    gain = balanced_gain(wl, mode)
    got, got_aux, ref, ref_aux, ex = _run(wl, FULL_PATH, mode, gain, want_state=True)
    S, z = oracle_state(wl, ex["data64"])
    assert errors(ex["S"], S)[0] <= 5e-3 and errors(ex["z"], z)[0] <= 5e-3
    ok = np.isfinite(ref).all(-1)
    assert ok.mean() > 0.99
    assert_parity(got[ok], ref[ok], _tag(name, FULL_PATH, mode, True))
    _check_aux(got_aux[ok], ref_aux[ok], wl, ex["n_softmax"])
    if wl.rate not in (0, 1):
        lam = np.exp(-ref_aux[..., 0]) if mode == O.STAB_EXACT else 1.0
        ratio = np.median((lam * ref_aux[..., 2] / ref_aux[..., 1])[ok])
        assert 0.2 < ratio < 5.0          # both branches carry weight


def test_two_layer_needs_its_second_weights_and_the_tensor_path():
    from paper_2509_24899_b200 import HybridAttention, binding, AsError, AS_PATH_SIMT
    wl = TWO_LAYER["two_layer_d128"]
    with pytest.raises(AsError) as e:
        HybridAttention.from_workload(wl, kernel_path=AS_PATH_SIMT)
    assert e.value.status == binding.AS_ERR_UNSUPPORTED
    op = HybridAttention.from_workload(wl)
    dev = {k: to_cuda_bf16(v) for k, v in W.generate(wl).items()}
    with pytest.raises(AsError) as e:
        op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"])
    assert e.value.status == binding.AS_ERR_INVALID_ARG
    with pytest.raises(AsError) as e:          # a bias that is not 4-byte aligned
        op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"], wq2=dev["wq2"], wk2=dev["wk2"],
                   biases={"bq1": dev["wq"].view(-1)[1:]})
    assert e.value.status == binding.AS_ERR_INVALID_ARG


def test_host_entry_point_pipelined_over_runs_of_heads():
    """Large enough that the host entry point works in several runs of heads (copies in, kernels and
    copies out overlapped): same bits as the device entry point, and the linear state of every head is
    in place afterwards."""
    import torch
    from paper_2509_24899_b200 import HybridAttention
    wl = W.Workload("host_runs", B=2, H=3, d=128, F=128, grid=(4, 64, 64), block=(2, 4, 4), rate=8, seed=21)
    data = W.generate(wl, wq_gain=0.02)
    dev = {k: to_cuda_bf16(v) for k, v in data.items()}
    op = HybridAttention.from_workload(wl, kernel_path=_path(FULL_PATH))
    ref = op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"]).clone()
    S_ref, z_ref = (t.clone() for t in op.linear_state())
    host = {k: torch.from_numpy(data[k].view(np.int16)).pin_memory() for k in ("q", "k", "v")}
    out_host = torch.zeros_like(host["q"]).pin_memory()
    for _ in range(2):                                   # the second call reuses the side streams and events
        out_host.zero_()
        op.forward_host(host["q"], host["k"], host["v"], dev["wq"], dev["wk"], out_host)
        torch.cuda.synchronize()
        assert op.last_status() == 0
        assert torch.equal(out_host, ref.view(torch.int16).cpu())
        S, z = op.linear_state()
        assert torch.equal(S, S_ref) and torch.equal(z, z_ref)


# More (batch, head) pairs than SMs, so that a persistent CTA walks over several units, with key loops of
# one, two and three tiles and with / without the linear tail: the hand-overs at unit boundaries (Q tile
# release, score columns, P tile, output accumulator) all happen with barrier phases that run on.
MANY_UNITS = {
    "one_key_tile_softmax_only": W.Workload("u1", B=2, H=80, d=128, F=128, grid=(1, 5, 7), block=(1, 5, 7), rate=1, seed=31),
    "two_key_tiles_softmax_only": W.Workload("u2", B=2, H=80, d=128, F=128, grid=(1, 10, 20), block=(1, 10, 20), rate=1, seed=32),
    "one_key_tile_hybrid": W.Workload("u3", B=2, H=80, d=128, F=128, grid=(1, 10, 30), block=(1, 5, 6), rate=3, seed=33),
    "three_key_tiles_hybrid_d64": W.Workload("u4", B=3, H=60, d=64, F=64, grid=(2, 12, 25), block=(1, 4, 5), rate=2, seed=34,
                                             rms_norm_qk=False),
    "no_key_tile_linear_only": W.Workload("u5", B=2, H=80, d=128, F=128, grid=(1, 10, 30), block=(1, 5, 6), rate=0, seed=35),
}


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("name", sorted(MANY_UNITS))
def test_many_units_per_cta(mode, name):
    wl = MANY_UNITS[name]
    gain = balanced_gain(wl, mode)
    got, got_aux, ref, ref_aux, ex = _run(wl, FULL_PATH, mode, gain)
    assert_parity(got, ref, _tag(name, FULL_PATH, mode, True))
    _check_aux(got_aux, ref_aux, wl, ex["n_softmax"])


# Layers without softmax tokens, one-layer map with F = d = 128: the streaming form of the query stage.  The cases
# cover how its runs of 128-row tiles are dealt to the CTAs: fewer tiles than SMs, heads that get one or two CTAs
# each, more heads than SMs (runs that cross heads: W and S are replaced on the way), a ragged last tile, degree 1.
STREAMING = {
    "few_tiles": W.Workload("s1", B=1, H=2, d=128, F=128, grid=(1, 10, 30), block=(1, 5, 6), rate=0, seed=41),
    "one_or_two_ctas_per_head": W.Workload("s2", B=2, H=50, d=128, F=128, grid=(1, 10, 25), block=(1, 5, 5), rate=0, seed=42),
    "more_heads_than_sms_degree1": W.Workload("s3", B=3, H=60, d=128, F=128, grid=(1, 10, 30), block=(1, 5, 6), rate=0, seed=43,
                                              degree=1),
    "long_runs": W.Workload("s4", B=1, H=1, d=128, F=128, grid=(8, 30, 52), block=(1, 6, 8), rate=0, seed=44),
}


@pytest.mark.parametrize("name", sorted(STREAMING))
def test_layers_without_softmax_tokens_streaming_form(name):
    wl = STREAMING[name]
    got, got_aux, ref, ref_aux, ex = _run(wl, FULL_PATH, O.STAB_PAPER, want_state=True)
    assert ex["n_softmax"] == 0
    ok = np.isfinite(ref).all(-1)          # a query with all-zero features is NaN in both
    assert ok.mean() > 0.99
    assert_parity(got[ok], ref[ok], _tag("streaming/" + name, FULL_PATH, O.STAB_PAPER))
    _check_aux(got_aux[ok], ref_aux[ok], wl, 0)
