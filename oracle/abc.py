"""ABC, the ungated ancestor of GSA (Eq. 3 and Eq. 4 of arXiv 2409.07146; the "no decay" row of the
table of ablations) -- TEST INFRASTRUCTURE ONLY.  Plain torch fp64, one token at a time:

    phi_t = exp(s_t) / sum_{j<=t} exp(s_j)                    (cumulative softmax over time, per slot)
    K~_t  = K~_{t-1} + phi_t (x) k_t,   V~_t = V~_{t-1} + phi_t (x) v_t
    o_t   = V~_t^T softmax(scale K~_t q_t)

Written with torch tensors so that autograd of this very definition gives the gradients.
"""
from __future__ import annotations

import numpy as np
import torch


def abc_forward(q, k, v, s, scale=1.0, K0=None, V0=None):
    """q,k [B,T,H,d_k], v [B,T,H,d_v], s [B,T,H,m] (score logits) as fp64 torch tensors.
    Returns (o [B,T,H,d_v], logits [B,T,H,m], K_T [B,H,m,d_k], V_T [B,H,m,d_v])."""
    B, T, H, dk = q.shape
    dv, m = v.shape[-1], s.shape[-1]
    K = torch.zeros(B, H, m, dk, dtype=torch.float64) if K0 is None else K0
    V = torch.zeros(B, H, m, dv, dtype=torch.float64) if V0 is None else V0
    Z = torch.zeros(B, H, m, dtype=torch.float64)
    outs, logits = [], []
    for t in range(T):
        e = torch.exp(s[:, t])                                   # [B,H,m]
        Z = Z + e
        phi = e / Z
        K = K + phi[..., None] * k[:, t][:, :, None, :]
        V = V + phi[..., None] * v[:, t][:, :, None, :]
        z = scale * torch.einsum("bhmd,bhd->bhm", K, q[:, t])
        p = torch.softmax(z, dim=-1)
        outs.append(torch.einsum("bhm,bhmd->bhd", p, V))
        logits.append(z)
    return torch.stack(outs, 1), torch.stack(logits, 1), K, V


def fwd(q, k, v, s, scale=1.0, K0=None, V0=None):
    t = lambda a: None if a is None else torch.tensor(np.asarray(a, dtype=np.float64))
    o, ok, KT, VT = abc_forward(t(q), t(k), t(v), t(s), scale, t(K0), t(V0))
    return dict(o=o.numpy(), ok=ok.numpy(), KT=KT.numpy(), VT=VT.numpy())


def bwd(q, k, v, s, dO, scale=1.0, K0=None, V0=None):
    """Gradients of sum(o * dO) by autograd of abc_forward: dict(dq, dk, dv, dgate (w.r.t. s), dK0, dV0)."""
    t = lambda a: None if a is None else torch.tensor(np.asarray(a, dtype=np.float64), requires_grad=True)
    qt, kt, vt, st, K0t, V0t = t(q), t(k), t(v), t(s), t(K0), t(V0)
    o, _, _, _ = abc_forward(qt, kt, vt, st, scale, K0t, V0t)
    (o * torch.tensor(np.asarray(dO, dtype=np.float64))).sum().backward()
    g = lambda x: None if x is None else x.grad.numpy()
    return dict(dq=g(qt), dk=g(kt), dv=g(vt), dgate=g(st), dK0=g(K0t), dV0=g(V0t))
