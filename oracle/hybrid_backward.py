"""Float64 CPU oracle for the gradient of the value-distillation loss w.r.t. the feature-map weights
(test infrastructure).

This module is TEST INFRASTRUCTURE, like `oracle/hybrid_attention.py`, whose forward pass it builds
on; it shares no code with the CUDA path and never imports it.

What it follows (paper: "Attention Surgery", arXiv 2509.24899):

* The value-distillation loss of section "Attention Distillation" (label `eq:vd_loss`):
  L = || y - y_hat ||_1, with y the teacher block's output and y_hat the hybrid attention output.
* Algorithm 1 (attention distillation): the student's update touches the parameters of phi only, so
  the gradient asked for is dL/dW_q and dL/dW_k of every head; q, k, v and the teacher output are
  constants of the step.

The gradient of a composition has a plain definition - the chain rule - and that is what is written
out here, step by step in the order of the forward pass run backwards.  For one (batch, head), with
one-layer feature maps a = W x, r = ReLU(a), phi = r^p elementwise (p the power of the feature's
part), softmax tokens T_S and linear tokens T_L:

    y_hat_i = num_i / den_i,   num_i = N_i + lambda_i phi_q,i S,   den_i = D_i + lambda_i phi_q,i . z
    S = sum_{j in T_L} phi_k,j^T v_j,   z = sum_{j in T_L} phi_k,j

N_i, D_i (the softmax branch) and lambda_i (1, or exp(-c_i)) do not depend on the weights.

    G_i       = dL/dy_hat_i  = sign(y_hat_i - y_i)
    dL/dnum_i = G_i / den_i                      =: g_i          [d]
    dL/dden_i = -(G_i . y_hat_i) / den_i         =: s_i          scalar
    dL/dphi_q,i = lambda_i (S g_i + z s_i)                       [F]
    dL/dS     = sum_i lambda_i phi_q,i^T g_i                     [F, d]
    dL/dz     = sum_i lambda_i phi_q,i s_i                       [F]
    dL/dphi_k,j = (dL/dS) v_j + dL/dz            for j in T_L    [F]
    dL/da     = dL/dphi * p r^(p-1) * [a > 0]
    dL/dW_q   = sum_i (dL/da_q,i)^T q_i,   dL/dW_k = sum_{j in T_L} (dL/da_k,j)^T k_j          [F, d]

The L1 norm is not differentiable where y_hat = y; sign(0) = 0 is taken there (a set of measure zero
for real-valued inputs).  Scope: one-layer feature maps without bias (what the CUDA path implements);
deeper maps follow the same rule with one more factor per layer.
"""
from __future__ import annotations


import numpy as np

from oracle import hybrid_attention as O


def value_distillation_loss(y_student, y_teacher):
    """|| y - y_hat ||_1 summed over every element ("Attention Distillation", value-distillation loss)."""
    return float(np.abs(np.asarray(y_teacher, dtype=np.float64) - np.asarray(y_student, dtype=np.float64)).sum())


def _powers(F, degree):
    part = F // degree
    return np.repeat(np.arange(1, degree + 1), part).astype(np.float64)        # p(f) per feature


def phi_weight_gradients_head(q, k, v, wq, wk, is_softmax, y_teacher, scale=None, stab_mode=O.STAB_PAPER, degree=2):
    """One (batch, head).  q, k, v, y_teacher: [N, d]; wq, wk: [F, d] (one layer, no bias).

    Returns (loss, dWq [F, d], dWk [F, d]): the value-distillation loss of this head's output and its
    gradient w.r.t. the two weight matrices."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    wq = np.asarray(wq, dtype=np.float64)
    wk = np.asarray(wk, dtype=np.float64)
    y = np.asarray(y_teacher, dtype=np.float64)
    mask = np.asarray(is_softmax, dtype=bool)
    N, d = q.shape
    F = wq.shape[0]
    lin = ~mask
    # forward, keeping what the chain rule needs
    y_hat, aux = O.hybrid_attention_head(q, k, v, wq, wk, mask, scale, stab_mode, degree)
    loss = value_distillation_loss(y_hat, y)
    dWq = np.zeros((F, d))
    dWk = np.zeros((F, d))
    if not lin.any():
        return loss, dWq, dWk                      # no linear tokens: the output does not depend on phi
    p = _powers(F, degree)
    a_q = q @ wq.T                                 # [N, F]
    r_q = np.maximum(a_q, 0.0)
    phi_q = r_q ** p
    a_k = k[lin] @ wk.T                            # [N_L, F]
    r_k = np.maximum(a_k, 0.0)
    phi_k = r_k ** p
    S = phi_k.T @ v[lin]                           # [F, d]
    z = phi_k.sum(axis=0)                          # [F]
    lam = np.ones(N)
    if mask.any() and stab_mode == O.STAB_EXACT:
        lam = np.exp(-aux[:, 0])
    den = aux[:, 1] + lam * aux[:, 2]              # D_i + lambda_i phi_q,i . z
    # backwards
    G = np.sign(y_hat - y)                         # dL/dy_hat
    g = G / den[:, None]                           # dL/dnum
    s = -(G * y_hat).sum(axis=1) / den             # dL/dden
    d_phi_q = lam[:, None] * (g @ S.T + s[:, None] * z[None, :])
    dS = (lam[:, None] * phi_q).T @ g
    dz = (lam[:, None] * phi_q).T @ s
    d_phi_k = v[lin] @ dS.T + dz[None, :]
    with np.errstate(divide="ignore", invalid="ignore"):
        slope_q = np.where(a_q > 0.0, p * r_q ** (p - 1.0), 0.0)
        slope_k = np.where(a_k > 0.0, p * r_k ** (p - 1.0), 0.0)
    dWq = (d_phi_q * slope_q).T @ q
    dWk = (d_phi_k * slope_k).T @ k[lin]
    return loss, dWq, dWk


def phi_weight_gradients(q, k, v, wq, wk, is_softmax, y_teacher, scale=None, stab_mode=O.STAB_PAPER, degree=2):
    """All (batch, head) pairs.  q, k, v, y_teacher: [B, H, N, d]; wq, wk: [H, F, d].

    Returns (loss, dWq [H, F, d], dWk [H, F, d]): the loss summed over everything, the gradients summed
    over the batch (the weights are per head)."""
    q = np.asarray(q)
    B, H = q.shape[:2]
    dWq = np.zeros(np.asarray(wq).shape)
    dWk = np.zeros(np.asarray(wk).shape)
    loss = 0.0
    for b in range(B):
        for h in range(H):
            l, gq, gk = phi_weight_gradients_head(q[b, h], k[b, h], v[b, h], wq[h], wk[h], is_softmax,
                                                  y_teacher[b, h], scale, stab_mode, degree)
            loss += l
            dWq[h] += gq
            dWk[h] += gk
    return loss, dWq, dWk
