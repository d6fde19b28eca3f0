"""The allocation-free entry point against the regular one (collected last on purpose: a run that
stops at the first failure has then already run every other test).

`as_hybrid_attn_linear_state_static` serves callers that cannot obtain device memory: processes
whose arena already owns the whole GPU, plug-ins restricted to the buffers they are handed, loops
that must not pay cudaMalloc's device-wide synchronisation.  It keeps its partial sums in a fixed
array inside the library, so consecutive calls see each other's leftovers; the test therefore makes
several calls in a row, with different shapes, and checks each against the handle-based path
(forward + linear_state) and against the float64 oracle within the tolerance used for S and z
elsewhere in the suite, and that a call leaves the amount of free device memory as it was."""
import numpy as np
import pytest

from paper_2509_24899_b200 import workloads as W
from _util import errors, oracle_inputs, oracle_state, to_cuda_bf16

pytestmark = pytest.mark.gpu

CASES = [
    W.Workload("na_d128", B=1, H=2, d=128, F=128, grid=(3, 10, 13), block=(1, 6, 8), rate=4, seed=21),
    W.Workload("na_d64", B=2, H=3, d=64, F=64, grid=(2, 9, 31), block=(1, 4, 4), rate=2, seed=22,
               rms_norm_qk=False),
    W.Workload("na_d128", B=1, H=2, d=128, F=128, grid=(3, 10, 13), block=(1, 6, 8), rate=4, seed=21),
    W.Workload("na_lin", B=1, H=1, d=128, F=128, grid=(2, 30, 52), block=(1, 6, 8), rate=0, seed=23),
    # at the size limit: one partial per (batch, head) fills the array almost completely, z sits at its very end
    W.Workload("na_limit_d128", B=1, H=127, d=128, F=128, grid=(1, 6, 11), block=(1, 3, 4), rate=3, seed=24),
    W.Workload("na_limit_d64", B=8, H=63, d=64, F=64, grid=(1, 5, 9), block=(1, 5, 3), rate=2, seed=25, rms_norm_qk=False),
]


def _static_state(wl, dev):
    import torch
    from paper_2509_24899_b200 import binding
    S = torch.full((wl.B, wl.H, wl.F, wl.d), float("nan"), dtype=torch.float32, device="cuda")
    z = torch.full((wl.B, wl.H, wl.F), float("nan"), dtype=torch.float32, device="cuda")
    binding.as_hybrid_attn_linear_state_static(
        dev["k"].data_ptr(), dev["v"].data_ptr(), dev["wk"].data_ptr(), wl.B, wl.H, wl.N, wl.d,
        wl.grid, wl.block, wl.rate, wl.degree, S.data_ptr(), z.data_ptr(),
        torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return S.cpu().numpy().astype(np.float64), z.cpu().numpy().astype(np.float64)


def _handle_state(wl, dev, path):
    import torch
    from paper_2509_24899_b200 import HybridAttention
    op = HybridAttention.from_workload(wl, kernel_path=path)
    op.forward(dev["q"], dev["k"], dev["v"], dev["wq"], dev["wk"])
    S, z = op.linear_state()
    torch.cuda.synchronize()
    assert op.last_status() == 0
    return S.cpu().numpy().astype(np.float64), z.cpu().numpy().astype(np.float64)


def test_static_linear_state_matches_handle_path_on_consecutive_calls():
    import torch
    from paper_2509_24899_b200 import AS_PATH_SIMT, AS_PATH_TENSOR
    for i, wl in enumerate(CASES):                      # back to back: the scratch array is reused
        data = W.generate(wl)
        dev = {k: to_cuda_bf16(v) for k, v in data.items()}
        S, z = _static_state(wl, dev)
        assert np.isfinite(S).all() and np.isfinite(z).all()
        S_or, z_or = oracle_state(wl, oracle_inputs(data))
        assert errors(S, S_or)[0] <= 5e-3 and errors(z, z_or)[0] <= 5e-3, wl.name
        if i > 0:
            # not the first call on the device: the entry point must not take or give back device memory
            # (the outputs are allocated before the measurement, by the caching allocator of the test itself)
            out_S = torch.empty((wl.B, wl.H, wl.F, wl.d), dtype=torch.float32, device="cuda")
            out_z = torch.empty((wl.B, wl.H, wl.F), dtype=torch.float32, device="cuda")
            torch.cuda.synchronize()
            free0 = torch.cuda.mem_get_info()[0]
            from paper_2509_24899_b200 import binding
            binding.as_hybrid_attn_linear_state_static(
                dev["k"].data_ptr(), dev["v"].data_ptr(), dev["wk"].data_ptr(), wl.B, wl.H, wl.N, wl.d, wl.grid,
                wl.block, wl.rate, wl.degree, out_S.data_ptr(), out_z.data_ptr(), torch.cuda.current_stream().cuda_stream)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free0, wl.name
        for path in (AS_PATH_SIMT, AS_PATH_TENSOR):
            S_ref, z_ref = _handle_state(wl, dev, path)
            assert errors(S, S_ref)[0] <= 5e-3, (wl.name, path)
            assert errors(z, z_ref)[0] <= 5e-3, (wl.name, path)


def test_static_linear_state_rejects_sizes_beyond_its_array():
    import torch
    from paper_2509_24899_b200 import binding, AsError
    t = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    o = torch.zeros(16, dtype=torch.float32, device="cuda")
    with pytest.raises(AsError) as e:                  # 128 heads x 128 x 129 floats > 8 MiB: nothing is launched
        binding.as_hybrid_attn_linear_state_static(t.data_ptr(), t.data_ptr(), t.data_ptr(), 1, 128, 64, 128,
                                                   (1, 8, 8), (1, 8, 8), 8, 2, o.data_ptr(), o.data_ptr(), 0)
    assert e.value.status == binding.AS_ERR_UNSUPPORTED
    with pytest.raises(AsError) as e:                  # grid product != N
        binding.as_hybrid_attn_linear_state_static(t.data_ptr(), t.data_ptr(), t.data_ptr(), 1, 1, 65, 128,
                                                   (1, 8, 8), (1, 8, 8), 8, 2, o.data_ptr(), o.data_ptr(), 0)
    assert e.value.status == binding.AS_ERR_INVALID_ARG
    torch.cuda.synchronize()
