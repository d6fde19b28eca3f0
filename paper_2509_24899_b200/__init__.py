"""B200-native hybrid attention forward (Attention Surgery, arXiv 2509.24899).

`binding` mirrors the C ABI one to one; `HybridAttention` is a small convenience wrapper that
lets PyTorch own the device memory and the stream.  All arithmetic runs in the CUDA library.
"""
from __future__ import annotations

from . import binding
from .binding import (AS_PATH_SIMT, AS_PATH_TENSOR, AS_STAB_EXACT, AS_STAB_PAPER, AsError)
from .binding import as_select_block_rates as select_block_rates

__all__ = ["binding", "HybridAttention", "AS_PATH_SIMT", "AS_PATH_TENSOR", "AS_STAB_EXACT",
           "AS_STAB_PAPER", "AsError", "select_block_rates"]


class HybridAttention:
    """One layer geometry bound to the current CUDA device.

    q, k, v: torch.bfloat16 CUDA tensors [B, H, N, d]; wq, wk: bfloat16 [H, F, d]; with phi_layers=2 the
    feature map is relu(relu(x wq^T + bq1) wq2^T + bq2) before the powers, wq, wk: [H, hidden, d], wq2, wk2:
    bfloat16 [H, F, hidden].  Biases (optional, bfloat16 [H, width]) are passed as `biases={"bq1": t, ...}`.
    """

    def __init__(self, B, H, N, d, grid, block, rate, phi_dim=None, poly_degree=2, softmax_scale=0.0,
                 stab_mode=AS_STAB_PAPER, kernel_path=AS_PATH_TENSOR, softmax_idx=None, phi_layers=1, phi_hidden=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("HybridAttention needs a CUDA device; there is no CPU fallback")
        self.shape = (B, H, N, d)
        self.F = d if phi_dim is None else phi_dim
        self.rate = rate
        self._desc = binding.make_desc(B, H, N, d, grid, block, rate, phi_dim, poly_degree, softmax_scale,
                                       stab_mode, kernel_path, softmax_idx, phi_layers=phi_layers,
                                       phi_hidden=(phi_hidden or self.F) if phi_layers == 2 else 0)
        self._h = binding.as_hybrid_attn_create(self._desc)
        self.workspace_bytes = binding.as_hybrid_attn_workspace_bytes(self._h)
        self.workspace_bytes_host = binding.as_hybrid_attn_workspace_bytes_host(self._h)
        self.n_softmax, _ = binding.as_hybrid_attn_softmax_tokens(self._h, want_indices=False)
        self._ws = None

    @classmethod
    def from_workload(cls, wl, **kw):
        return cls(wl.B, wl.H, wl.N, wl.d, wl.grid, wl.block, wl.rate, phi_dim=wl.F,
                   poly_degree=wl.degree, phi_layers=wl.layers, phi_hidden=wl.hidden_width, **kw)

    @property
    def handle(self):
        return self._h

    def workspace(self, host: bool = False):
        import torch
        need = self.workspace_bytes_host if host else self.workspace_bytes
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device="cuda")
        return self._ws

    def softmax_indices(self):
        return binding.as_hybrid_attn_softmax_tokens(self._h)[1]

    def forward(self, q, k, v, wq=None, wk=None, out=None, aux=None, stream=None, wq2=None, wk2=None,
                workspace=None, biases=None):
        """`workspace` (optional): a caller-owned uint8 CUDA tensor of at least `workspace_bytes`, 256-byte
        aligned; it becomes the handle's workspace for `linear_state` as well."""
        import torch
        if out is None:
            out = torch.empty_like(q)
        if workspace is not None:
            self._ws = workspace
        ws = self.workspace()
        st = torch.cuda.current_stream() if stream is None else stream
        binding.as_hybrid_attn_forward(
            self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(),
            0 if wq is None else wq.data_ptr(), 0 if wk is None else wk.data_ptr(),
            out.data_ptr(), 0 if aux is None else aux.data_ptr(), ws.data_ptr(), ws.numel(), st.cuda_stream,
            0 if wq2 is None else wq2.data_ptr(), 0 if wk2 is None else wk2.data_ptr(),
            None if biases is None else {n: t.data_ptr() for n, t in biases.items()})
        return out

    def forward_host(self, q_host, k_host, v_host, wq, wk, out_host, stream=None, wq2=None, wk2=None, biases=None):
        """q_host, k_host, v_host, out_host: pinned CPU tensors; the weights are device tensors."""
        import torch
        ws = self.workspace(host=True)
        st = torch.cuda.current_stream() if stream is None else stream
        binding.as_hybrid_attn_forward_host(
            self._h, q_host.data_ptr(), k_host.data_ptr(), v_host.data_ptr(),
            0 if wq is None else wq.data_ptr(), 0 if wk is None else wk.data_ptr(),
            out_host.data_ptr(), ws.data_ptr(), ws.numel(), st.cuda_stream,
            0 if wq2 is None else wq2.data_ptr(), 0 if wk2 is None else wk2.data_ptr(),
            None if biases is None else {n: t.data_ptr() for n, t in biases.items()})
        return out_host

    def key_pass(self, k, v, wq=None, wk=None, stream=None, wq2=None, wk2=None, biases=None):
        """First stage of a sequence-sharded forward on this handle's token range.  Returns (K_S, V_S, S, z): the
        range's softmax keys / values [B*H, n_softmax, d] (bf16) and its partial linear state [B*H, F, d], [B*H, F]
        (fp32).  K_S, V_S, S, z are views into the handle's workspace (k, v themselves and zeros for a range without
        linear tokens)."""
        import torch
        B, H, N, d = self.shape
        BH = B * H
        if self.n_softmax == N:
            return (k.reshape(BH, N, d), v.reshape(BH, N, d),
                    torch.zeros(BH, self.F, d, dtype=torch.float32, device=k.device),
                    torch.zeros(BH, self.F, dtype=torch.float32, device=k.device))
        ws = self.workspace()
        st = torch.cuda.current_stream() if stream is None else stream
        binding.as_hybrid_attn_key_pass(
            self._h, k.data_ptr(), v.data_ptr(), 0 if wq is None else wq.data_ptr(), 0 if wk is None else wk.data_ptr(),
            ws.data_ptr(), ws.numel(), st.cuda_stream, 0 if wq2 is None else wq2.data_ptr(),
            0 if wk2 is None else wk2.data_ptr(), None if biases is None else {n: t.data_ptr() for n, t in biases.items()})
        o_ks, o_vs, o_S, o_z = binding.as_hybrid_attn_workspace_offsets(self._h)
        n_s = self.n_softmax
        view = lambda off, count, dtype, shape: ws[off:off + count * dtype.itemsize].view(dtype).view(*shape)
        ks = view(o_ks, BH * n_s * d, torch.bfloat16, (BH, n_s, d))
        vs = view(o_vs, BH * n_s * d, torch.bfloat16, (BH, n_s, d))
        return ks, vs, view(o_S, BH * self.F * d, torch.float32, (BH, self.F, d)), view(o_z, BH * self.F, torch.float32, (BH, self.F))

    def query_pass(self, q, wq, wk, ks, vs, S, z, out=None, aux=None, stream=None, wq2=None, wk2=None, biases=None):
        """Second stage: this range's queries against the gathered softmax keys ks, vs [B*H, n_keys, d] and the summed
        state S, z (None, None when the layer has no linear tokens).  Returns the range's output rows."""
        import torch
        if out is None:
            out = torch.empty_like(q)
        ws = self.workspace()
        st = torch.cuda.current_stream() if stream is None else stream
        n_keys = 0 if ks is None else ks.shape[1]
        binding.as_hybrid_attn_query_pass(
            self._h, q.data_ptr(), 0 if wq is None else wq.data_ptr(), 0 if wk is None else wk.data_ptr(),
            ks.data_ptr() if n_keys else 0, vs.data_ptr() if n_keys else 0, n_keys,
            0 if S is None else S.data_ptr(), 0 if z is None else z.data_ptr(), out.data_ptr(),
            0 if aux is None else aux.data_ptr(), ws.data_ptr(), ws.numel(), st.cuda_stream,
            0 if wq2 is None else wq2.data_ptr(), 0 if wk2 is None else wk2.data_ptr(),
            None if biases is None else {n: t.data_ptr() for n, t in biases.items()})
        return out

    def backward_phi(self, q, k, v, wq, wk, y_teacher, y_hat, aux, stream=None, want_loss=True):
        """(dWq, dWk, loss) of the value-distillation loss sum |y_teacher - y_hat| w.r.t. the feature-map weights,
        after `forward(..., out=y_hat, aux=aux)` on the same inputs (the handle's workspace still holds S and z)."""
        import torch
        B, H, N, d = self.shape
        dwq = torch.empty(H, self.F, d, dtype=torch.float32, device="cuda")
        dwk = torch.empty_like(dwq)
        loss = torch.zeros(1, dtype=torch.float32, device="cuda") if want_loss else None
        need = binding.as_hybrid_attn_backward_workspace_bytes(self._h)
        if getattr(self, "_bws", None) is None or self._bws.numel() < need:
            self._bws = torch.empty(need, dtype=torch.uint8, device="cuda")
        st = torch.cuda.current_stream() if stream is None else stream
        binding.as_hybrid_attn_backward_phi(
            self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), wq.data_ptr(), wk.data_ptr(), y_teacher.data_ptr(),
            y_hat.data_ptr(), aux.data_ptr(), self.workspace().data_ptr(), dwq.data_ptr(), dwk.data_ptr(),
            0 if loss is None else loss.data_ptr(), self._bws.data_ptr(), self._bws.numel(), st.cuda_stream)
        return dwq, dwk, loss

    def linear_state(self, stream=None):
        """(S [B,H,F,d], z [B,H,F]) fp32 as left in the workspace by the last forward."""
        import torch
        B, H, N, d = self.shape
        S = torch.empty(B, H, self.F, d, dtype=torch.float32, device="cuda")
        z = torch.empty(B, H, self.F, dtype=torch.float32, device="cuda")
        st = torch.cuda.current_stream() if stream is None else stream
        binding.as_hybrid_attn_linear_state(self._h, self.workspace().data_ptr(), S.data_ptr(), z.data_ptr(),
                                            st.cuda_stream)
        return S, z

    def last_status(self, stream=None) -> int:
        import torch
        st = torch.cuda.current_stream() if stream is None else stream
        return binding.as_hybrid_attn_last_status(self._h, st.cuda_stream)

    def close(self):
        if getattr(self, "_h", None) is not None:
            binding.as_hybrid_attn_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
