"""The C-ABI library loads, exports every symbol the header declares, and rejects bad
arguments on the host (no GPU needed: these paths return before any kernel launch)."""
import ctypes as C
import os
import re

import pytest

from paper_2509_24899_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def _declared_symbols():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            names += re.findall(r"AS_API[^;(]*?\b(as_[a-z0-9_]+)\s*\(", text)
    return names


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert len(names) >= 13 and "as_hybrid_attn_forward" in names
    for n in names:
        assert hasattr(lib, n), "symbol %s declared in include/ but not exported" % n


def test_binding_mirrors_every_entry_point():
    for n in _declared_symbols():
        assert hasattr(binding, n), "binding lacks %s" % n


def test_status_strings(lib):
    seen = {binding.as_status_string(i) for i in range(8)}
    assert len(seen) == 8 and binding.as_status_string(0) == "ok"
    assert binding.as_status_string(99) == "unknown status"


def _desc(**kw):
    args = dict(B=1, H=2, N=1024, d=64, grid=(4, 16, 16), block=(2, 4, 4), rate=32)
    args.update(kw)
    return binding.make_desc(**args)


@pytest.mark.parametrize("kw,status", [
    (dict(N=1000), binding.AS_ERR_INVALID_ARG),                 # grid product != N
    (dict(B=0), binding.AS_ERR_INVALID_ARG),
    (dict(rate=-1), binding.AS_ERR_INVALID_ARG),
    (dict(block=(0, 4, 4)), binding.AS_ERR_INVALID_ARG),
    (dict(stab_mode=7), binding.AS_ERR_INVALID_ARG),
    (dict(softmax_scale=float("nan")), binding.AS_ERR_INVALID_ARG),
    (dict(softmax_idx=[3, 3]), binding.AS_ERR_INVALID_ARG),      # not strictly increasing
    (dict(softmax_idx=[5, 2000]), binding.AS_ERR_INVALID_ARG),   # out of range
    (dict(poly_degree=3), binding.AS_ERR_INVALID_ARG),           # 64 not divisible by 3
    (dict(d=96, phi_dim=96), binding.AS_ERR_UNSUPPORTED),
    (dict(phi_dim=192), binding.AS_ERR_UNSUPPORTED),             # neither d nor a multiple of 128
    (dict(phi_dim=640), binding.AS_ERR_UNSUPPORTED),             # more than 512 features
    (dict(poly_degree=4), binding.AS_ERR_UNSUPPORTED),           # parts of 16 features: not a multiple of 32
    (dict(phi_layers=2, phi_hidden=128), binding.AS_ERR_UNSUPPORTED),   # at d = 64 two layers need hidden = F = d
    (dict(d=128, phi_dim=256, phi_layers=2, phi_hidden=512), binding.AS_ERR_UNSUPPORTED),
    (dict(d=128, phi_dim=384, phi_layers=2, phi_hidden=128), binding.AS_ERR_UNSUPPORTED),
    (dict(phi_layers=3, phi_hidden=64), binding.AS_ERR_UNSUPPORTED),
    (dict(phi_dim=128, kernel_path=binding.AS_PATH_SIMT), binding.AS_ERR_UNSUPPORTED),   # the check path has F = d only
])
def test_create_rejects_bad_descriptors(lib, kw, status):
    h = C.c_void_p()
    d = _desc(**kw)
    assert lib.as_hybrid_attn_create(C.byref(d), C.byref(h)) == status
    assert h.value is None                                       # out-parameter untouched


def test_create_null_and_struct_size(lib):
    h = C.c_void_p()
    assert lib.as_hybrid_attn_create(None, C.byref(h)) == binding.AS_ERR_INVALID_ARG
    d = _desc()
    assert lib.as_hybrid_attn_create(C.byref(d), None) == binding.AS_ERR_INVALID_ARG
    d.struct_size = 8
    assert lib.as_hybrid_attn_create(C.byref(d), C.byref(h)) == binding.AS_ERR_INVALID_ARG


def test_null_handles_are_rejected_and_destroy_null_is_noop(lib):
    n = C.c_size_t()
    assert lib.as_hybrid_attn_destroy(None) == binding.AS_OK
    assert lib.as_hybrid_attn_workspace_bytes(None, C.byref(n)) == binding.AS_ERR_INVALID_ARG
    assert lib.as_hybrid_attn_forward(None, 0, 0, 0, None, 0, 0, 0, 0, 0) == binding.AS_ERR_INVALID_ARG
    assert lib.as_hybrid_attn_last_status(None, None) == binding.AS_ERR_INVALID_ARG


def test_create_without_a_device_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(binding.AsError) as e:
        binding.as_hybrid_attn_create(_desc())
    assert e.value.status in (binding.AS_ERR_CUDA, binding.AS_ERR_ARCH)
    from paper_2509_24899_b200 import HybridAttention
    with pytest.raises(RuntimeError):
        HybridAttention(1, 2, 1024, 64, (4, 16, 16), (2, 4, 4), 32)
