"""ctypes binding of libas_hybrid_attn: the same names as the C ABI, argument marshalling only.

Every step of the forward pass runs in the library's CUDA kernels.  PyTorch is used by the
callers for device memory and streams; this module passes raw pointers through.  If the shared
library is missing the import of any entry point raises - there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "lib", "libas_hybrid_attn.so")

AS_OK, AS_ERR_INVALID_ARG, AS_ERR_UNSUPPORTED, AS_ERR_ARCH = 0, 1, 2, 3
AS_ERR_ALLOC, AS_ERR_WORKSPACE, AS_ERR_CUDA, AS_ERR_DEVICE_TIMEOUT, AS_ERR_INFEASIBLE = 4, 5, 6, 7, 8
AS_STAB_PAPER, AS_STAB_EXACT = 0, 1
AS_ACT_RELU = 0
AS_PATH_TENSOR, AS_PATH_SIMT = 0, 1
AS_KERNEL_KPASS, AS_KERNEL_REDUCE, AS_KERNEL_QPASS, AS_NUM_KERNELS = 0, 1, 2, 3


class as_hybrid_attn_desc_t(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32),
        ("B", C.c_int32), ("H", C.c_int32), ("N", C.c_int32), ("d", C.c_int32),
        ("grid_t", C.c_int32), ("grid_h", C.c_int32), ("grid_w", C.c_int32),
        ("blk_t", C.c_int32), ("blk_h", C.c_int32), ("blk_w", C.c_int32),
        ("rate_den", C.c_int32),
        ("softmax_idx", C.POINTER(C.c_int32)),
        ("n_softmax", C.c_int32),
        ("phi_dim", C.c_int32), ("phi_layers", C.c_int32), ("phi_hidden", C.c_int32),
        ("poly_degree", C.c_int32), ("phi_act", C.c_int32),
        ("softmax_scale", C.c_float),
        ("stab_mode", C.c_int32),
        ("kernel_path", C.c_int32),
    ]


class as_phi_weights_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("wq1", "bq1", "wq2", "bq2", "wk1", "bk1", "wk2", "bk2")]


class AsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, as_status_string(status), status))


_lib = None


def lib() -> C.CDLL:
    """Loads the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libas_hybrid_attn.so is missing at %s; run "
                              "`python -m paper_2509_24899_b200.build` (needs nvcc)" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        H = C.c_void_p
        sigs = {
            "as_hybrid_attn_create": [C.POINTER(as_hybrid_attn_desc_t), C.POINTER(H)],
            "as_hybrid_attn_destroy": [H],
            "as_hybrid_attn_workspace_bytes": [H, C.POINTER(C.c_size_t)],
            "as_hybrid_attn_workspace_bytes_host": [H, C.POINTER(C.c_size_t)],
            "as_hybrid_attn_forward": [H, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(as_phi_weights_t),
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p],
            "as_hybrid_attn_forward_host": [H, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(as_phi_weights_t),
                                            C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p],
            "as_hybrid_attn_linear_state": [H, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p],
            "as_hybrid_attn_softmax_tokens": [H, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.c_int32],
            "as_hybrid_attn_last_status": [H, C.c_void_p],
            "as_hybrid_attn_debug_expire_wait": [H, C.c_int64, C.c_void_p],
            "as_hybrid_attn_key_pass": [H, C.c_void_p, C.c_void_p, C.POINTER(as_phi_weights_t), C.c_void_p, C.c_size_t, C.c_void_p],
            "as_hybrid_attn_workspace_offsets": [H] + [C.POINTER(C.c_size_t)] * 4,
            "as_hybrid_attn_query_pass": [H, C.c_void_p, C.POINTER(as_phi_weights_t), C.c_void_p, C.c_void_p, C.c_int32,
                                          C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p],
            "as_hybrid_attn_backward_workspace_bytes": [H, C.POINTER(C.c_size_t)],
            "as_hybrid_attn_backward_phi": [H, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(as_phi_weights_t), C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_size_t, C.c_void_p],
            "as_hybrid_attn_profile_enable": [H, C.c_int32],
            "as_hybrid_attn_profile_read": [H, C.POINTER(C.c_float), C.POINTER(C.c_int32)],
            "as_hybrid_attn_launch_count": [H, C.POINTER(C.c_uint64)],
            "as_hybrid_attn_linear_state_static": [C.c_void_p, C.c_void_p, C.c_void_p] + [C.c_int32] * 12
                                                  + [C.c_void_p, C.c_void_p, C.c_void_p],
            "as_select_block_rates": [C.c_int32, C.c_int32, C.POINTER(C.c_double), C.POINTER(C.c_double), C.c_double,
                                      C.POINTER(C.c_int32), C.POINTER(C.c_double), C.POINTER(C.c_double)],
        }
        for name, args in sigs.items():
            fn = getattr(L, name)
            fn.argtypes = args
            fn.restype = C.c_int
        L.as_status_string.argtypes = [C.c_int]
        L.as_status_string.restype = C.c_char_p
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != AS_OK:
        raise AsError(status, where)


def as_status_string(status: int) -> str:
    return lib().as_status_string(int(status)).decode()


def make_desc(B, H, N, d, grid, block, rate, phi_dim=None, poly_degree=2, softmax_scale=0.0,
              stab_mode=AS_STAB_PAPER, kernel_path=AS_PATH_TENSOR, softmax_idx=None,
              phi_layers=1, phi_hidden=0) -> as_hybrid_attn_desc_t:
    """Fills the descriptor struct; `softmax_idx` (optional) is a sequence of token indices."""
    desc = as_hybrid_attn_desc_t()
    desc.struct_size = C.sizeof(as_hybrid_attn_desc_t)
    desc.B, desc.H, desc.N, desc.d = B, H, N, d
    desc.grid_t, desc.grid_h, desc.grid_w = grid
    desc.blk_t, desc.blk_h, desc.blk_w = block
    desc.rate_den = rate
    if softmax_idx is not None:
        arr = (C.c_int32 * len(softmax_idx))(*[int(i) for i in softmax_idx])
        desc.softmax_idx = C.cast(arr, C.POINTER(C.c_int32))
        desc.n_softmax = len(softmax_idx)
        desc._keepalive = arr
    desc.phi_dim = d if phi_dim is None else phi_dim
    desc.phi_layers, desc.phi_hidden = phi_layers, phi_hidden
    desc.poly_degree, desc.phi_act = poly_degree, AS_ACT_RELU
    desc.softmax_scale = softmax_scale
    desc.stab_mode, desc.kernel_path = stab_mode, kernel_path
    return desc


def as_hybrid_attn_create(desc: as_hybrid_attn_desc_t) -> C.c_void_p:
    h = C.c_void_p()
    _check(lib().as_hybrid_attn_create(C.byref(desc), C.byref(h)), "as_hybrid_attn_create")
    return h


def as_hybrid_attn_destroy(h) -> None:
    _check(lib().as_hybrid_attn_destroy(h), "as_hybrid_attn_destroy")


def as_hybrid_attn_workspace_bytes(h) -> int:
    n = C.c_size_t()
    _check(lib().as_hybrid_attn_workspace_bytes(h, C.byref(n)), "as_hybrid_attn_workspace_bytes")
    return n.value


def as_hybrid_attn_workspace_bytes_host(h) -> int:
    n = C.c_size_t()
    _check(lib().as_hybrid_attn_workspace_bytes_host(h, C.byref(n)), "as_hybrid_attn_workspace_bytes_host")
    return n.value


def _weights(wq_ptr, wk_ptr, wq2_ptr=0, wk2_ptr=0, biases=None):
    """as_phi_weights_t from integer device addresses; `biases` maps 'bq1', 'bk1', 'bq2', 'bk2' to addresses."""
    if not wq_ptr and not wk_ptr:
        return None
    w = as_phi_weights_t()
    w.wq1, w.wk1 = wq_ptr, wk_ptr
    w.wq2, w.wk2 = wq2_ptr or None, wk2_ptr or None
    for name, ptr in (biases or {}).items():
        setattr(w, name, ptr or None)
    return C.byref(w)


def as_hybrid_attn_forward(h, q_ptr, k_ptr, v_ptr, wq_ptr, wk_ptr, out_ptr, aux_ptr, ws_ptr, ws_bytes,
                           stream_ptr, wq2_ptr=0, wk2_ptr=0, biases=None) -> None:
    """All pointers are integer device addresses (e.g. tensor.data_ptr()); 0 / None means NULL.
    wq2_ptr / wk2_ptr: second-layer weights of a two-layer feature map; biases: dict of addresses."""
    _check(lib().as_hybrid_attn_forward(h, q_ptr, k_ptr, v_ptr, _weights(wq_ptr, wk_ptr, wq2_ptr, wk2_ptr, biases), out_ptr,
                                        aux_ptr or None, ws_ptr, ws_bytes, stream_ptr or None), "as_hybrid_attn_forward")


def as_hybrid_attn_forward_host(h, q_host, k_host, v_host, wq_ptr, wk_ptr, out_host, ws_ptr, ws_bytes,
                                stream_ptr, wq2_ptr=0, wk2_ptr=0, biases=None) -> None:
    _check(lib().as_hybrid_attn_forward_host(h, q_host, k_host, v_host, _weights(wq_ptr, wk_ptr, wq2_ptr, wk2_ptr, biases),
                                             out_host, ws_ptr, ws_bytes, stream_ptr or None), "as_hybrid_attn_forward_host")


def as_hybrid_attn_linear_state(h, ws_ptr, S_ptr, z_ptr, stream_ptr) -> None:
    _check(lib().as_hybrid_attn_linear_state(h, ws_ptr, S_ptr or None, z_ptr or None, stream_ptr or None),
           "as_hybrid_attn_linear_state")


def as_hybrid_attn_softmax_tokens(h, want_indices: bool = True):
    """Returns (count, list of indices or None)."""
    n = C.c_int32()
    _check(lib().as_hybrid_attn_softmax_tokens(h, C.byref(n), None, 0), "as_hybrid_attn_softmax_tokens")
    if not want_indices:
        return n.value, None
    buf = (C.c_int32 * max(1, n.value))()
    _check(lib().as_hybrid_attn_softmax_tokens(h, C.byref(n), buf, n.value), "as_hybrid_attn_softmax_tokens")
    return n.value, list(buf[:n.value])


def as_hybrid_attn_last_status(h, stream_ptr) -> int:
    """Returns the status code instead of raising, so that callers can test for a time-out."""
    return lib().as_hybrid_attn_last_status(h, stream_ptr or None)


def as_hybrid_attn_key_pass(h, k_ptr, v_ptr, wq_ptr, wk_ptr, ws_ptr, ws_bytes, stream_ptr, wq2_ptr=0, wk2_ptr=0,
                            biases=None) -> None:
    """First stage of a sequence-sharded forward: this range's K_S, V_S and partial S, z into the workspace."""
    _check(lib().as_hybrid_attn_key_pass(h, k_ptr, v_ptr, _weights(wq_ptr, wk_ptr, wq2_ptr, wk2_ptr, biases), ws_ptr,
                                         ws_bytes, stream_ptr or None), "as_hybrid_attn_key_pass")


def as_hybrid_attn_workspace_offsets(h):
    """Byte offsets (K_S, V_S, S, z) inside the workspace."""
    o = [C.c_size_t() for _ in range(4)]
    _check(lib().as_hybrid_attn_workspace_offsets(h, *[C.byref(x) for x in o]), "as_hybrid_attn_workspace_offsets")
    return tuple(x.value for x in o)


def as_hybrid_attn_query_pass(h, q_ptr, wq_ptr, wk_ptr, ks_ptr, vs_ptr, n_keys, S_ptr, z_ptr, out_ptr, aux_ptr, ws_ptr,
                              ws_bytes, stream_ptr, wq2_ptr=0, wk2_ptr=0, biases=None) -> None:
    """Second stage: this range's queries against the gathered keys and the summed state."""
    _check(lib().as_hybrid_attn_query_pass(h, q_ptr, _weights(wq_ptr, wk_ptr, wq2_ptr, wk2_ptr, biases), ks_ptr or None,
                                           vs_ptr or None, int(n_keys), S_ptr or None, z_ptr or None, out_ptr,
                                           aux_ptr or None, ws_ptr, ws_bytes, stream_ptr or None),
           "as_hybrid_attn_query_pass")


def as_hybrid_attn_backward_workspace_bytes(h) -> int:
    n = C.c_size_t()
    _check(lib().as_hybrid_attn_backward_workspace_bytes(h, C.byref(n)), "as_hybrid_attn_backward_workspace_bytes")
    return n.value


def as_hybrid_attn_backward_phi(h, q_ptr, k_ptr, v_ptr, wq_ptr, wk_ptr, y_ptr, yhat_ptr, aux_ptr, fwd_ws_ptr, dwq_ptr,
                                dwk_ptr, loss_ptr, ws_ptr, ws_bytes, stream_ptr) -> None:
    """dL/dW_q, dL/dW_k (fp32 [H,F,d]) of L = sum |y - y_hat| after a forward; integer device addresses."""
    _check(lib().as_hybrid_attn_backward_phi(h, q_ptr, k_ptr, v_ptr, _weights(wq_ptr, wk_ptr), y_ptr, yhat_ptr, aux_ptr,
                                             fwd_ws_ptr, dwq_ptr, dwk_ptr, loss_ptr or None, ws_ptr, ws_bytes,
                                             stream_ptr or None), "as_hybrid_attn_backward_phi")


def as_hybrid_attn_debug_expire_wait(h, limit_cycles: int, stream_ptr) -> None:
    """Test aid: a kernel whose bounded wait runs out after `limit_cycles` SM clocks and sets the status word."""
    _check(lib().as_hybrid_attn_debug_expire_wait(h, int(limit_cycles), stream_ptr or None),
           "as_hybrid_attn_debug_expire_wait")


def as_hybrid_attn_profile_enable(h, enable: bool) -> None:
    _check(lib().as_hybrid_attn_profile_enable(h, 1 if enable else 0), "as_hybrid_attn_profile_enable")


def as_hybrid_attn_profile_read(h):
    """Returns (ms per kernel class, launches per kernel class) accumulated since the last read."""
    ms = (C.c_float * AS_NUM_KERNELS)()
    cnt = (C.c_int32 * AS_NUM_KERNELS)()
    _check(lib().as_hybrid_attn_profile_read(h, ms, cnt), "as_hybrid_attn_profile_read")
    return list(ms), list(cnt)


def as_hybrid_attn_launch_count(h) -> int:
    n = C.c_uint64()
    _check(lib().as_hybrid_attn_launch_count(h, C.byref(n)), "as_hybrid_attn_launch_count")
    return n.value


def as_hybrid_attn_linear_state_static(k_ptr, v_ptr, wk_ptr, B, H, N, d, grid, block, rate, poly_degree,
                                       S_ptr, z_ptr, stream_ptr) -> None:
    """S [B,H,d,d] and z [B,H,d] (fp32) of one layer without any allocation inside the library.

    For callers that cannot request device memory (an arena owns all of it, or only the buffers
    handed in may be used): no handle, no workspace; the partial sums use a fixed 8 MiB array inside
    the library.  Sizes beyond that array raise AsError(AS_ERR_UNSUPPORTED).  Calls must not overlap
    on the GPU; make the first call on a device outside any stream capture and before an arena takes the
    rest of the device's memory (the driver sets the array up when the library's code is first loaded on
    the device, which by default is that first call)."""
    _check(lib().as_hybrid_attn_linear_state_static(
        k_ptr, v_ptr, wk_ptr, B, H, N, d, grid[0], grid[1], grid[2], block[0], block[1], block[2], rate,
        poly_degree, S_ptr or None, z_ptr or None, stream_ptr or None), "as_hybrid_attn_linear_state_static")


def as_select_block_rates(cost, err, budget):
    """One rate index per block with minimal summed error under the cost budget.

    cost, err: [n_blocks][n_rates] (anything convertible to rows of floats).  Returns
    (choice: list of int, total_cost, total_err); raises AsError(AS_ERR_INFEASIBLE) when even the
    cheapest rates exceed the budget.  Host computation inside the library; no GPU is needed."""
    n_blocks = len(cost)
    n_rates = len(cost[0]) if n_blocks else 0
    if n_blocks == 0 or n_rates == 0 or len(err) != n_blocks or any(len(r) != n_rates for r in cost) \
            or any(len(r) != n_rates for r in err):
        raise AsError(AS_ERR_INVALID_ARG, "as_select_block_rates")
    flat_c = (C.c_double * (n_blocks * n_rates))(*[float(x) for row in cost for x in row])
    flat_e = (C.c_double * (n_blocks * n_rates))(*[float(x) for row in err for x in row])
    choice = (C.c_int32 * n_blocks)()
    tc, te = C.c_double(), C.c_double()
    _check(lib().as_select_block_rates(n_blocks, n_rates, flat_c, flat_e, float(budget), choice,
                                       C.byref(tc), C.byref(te)), "as_select_block_rates")
    return list(choice), tc.value, te.value
