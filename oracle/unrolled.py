"""Brute-force unrolled form of Gated Slot Attention -- TEST INFRASTRUCTURE ONLY.

A second statement of the layer, used by the CPU tests to pin the sequential
oracle on tiny inputs.  It evaluates the two-pass form of Eq. 7 (arXiv
2409.07146, Sec. 3.2) with every decay product written out explicitly:

    W[t, j, s]  = (1 - a_j[s]) * prod_{r=j+1..t} a_r[s]          (j <= t)
    D0[t, s]    = prod_{r=1..t} a_r[s]
    o'_t[s]     = scale * ( D0[t,s] <K0[s], q_t> + sum_{j<=t} <q_t, k_j> W[t,j,s] )
    p_t         = softmax_s(o'_t)
    o_t         = sum_s p_t[s] ( D0[t,s] V0[s] + sum_{j<=t} W[t,j,s] v_j )

No recurrence and no state is carried: cost O(T^2 m d) with O(T^3) products,
which is the point.  Written with torch CPU float64 ops so that autograd gives
an independent derivative of the same definition for the backward pins.
"""
from __future__ import annotations

import torch


def _slot_weights(logits, act):
    """softmax over the slots (Eq. 6) or its element-wise replacements in the paper's ablation
    on the non-linearity, each by the library's own routine."""
    if act == "softmax":
        return torch.softmax(logits, dim=-1)
    if act == "none":
        return logits
    if act == "relu":
        return torch.nn.functional.relu(logits)
    if act == "swish":
        return torch.nn.functional.silu(logits)
    if act == "relu2":
        return torch.nn.functional.relu(logits).square()
    raise ValueError(act)


def gsa_unrolled(q, k, v, a, K0=None, V0=None, scale=1.0, act="softmax"):
    """One head.  q,k [T,d_k]; v [T,d_v]; a [T,m] linear gate in [0,1];
    K0 [m,d_k], V0 [m,d_v] or None.  Returns (o [T,d_v], logits [T,m],
    K_T [m,d_k], V_T [m,d_v]) as float64 torch tensors (differentiable)."""
    q, k, v, a = (torch.as_tensor(x, dtype=torch.float64) for x in (q, k, v, a))
    T, m = a.shape
    rows_W, rows_D0 = [], []
    for t in range(T):
        row = []
        for j in range(T):
            if j <= t:
                w = 1.0 - a[j]
                for r in range(j + 1, t + 1):
                    w = w * a[r]
            else:
                w = torch.zeros(m, dtype=torch.float64)
            row.append(w)
        rows_W.append(torch.stack(row))
        d0 = torch.ones(m, dtype=torch.float64)
        for r in range(t + 1):
            d0 = d0 * a[r]
        rows_D0.append(d0)
    W = torch.stack(rows_W)            # [T(t), T(j), m]
    D0 = torch.stack(rows_D0)          # [T, m]
    P = q @ k.T                        # [T(t), T(j)]  <q_t, k_j>
    logits = torch.einsum("tj,tjs->ts", P, W)
    Kmem = torch.einsum("tjs,jc->tsc", W, k)      # K~_t for every t
    Vmem = torch.einsum("tjs,jc->tsc", W, v)
    if K0 is not None:
        K0 = torch.as_tensor(K0, dtype=torch.float64)
        logits = logits + D0 * (q @ K0.T)
        Kmem = Kmem + D0[:, :, None] * K0[None]
    if V0 is not None:
        V0 = torch.as_tensor(V0, dtype=torch.float64)
        Vmem = Vmem + D0[:, :, None] * V0[None]
    logits = scale * logits
    p = _slot_weights(logits, act)
    o = torch.einsum("ts,tsc->tc", p, Vmem)
    return o, logits, Kmem[-1], Vmem[-1]
