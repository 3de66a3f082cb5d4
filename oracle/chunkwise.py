"""Chunkwise-parallel form of Gated Slot Attention in fp64 -- TEST INFRASTRUCTURE ONLY.

A third statement of the layer, used by the CPU tests to check that the
chunkwise regrouping of Algorithm 1 (arXiv 2409.07146, App. A/B) reproduces the
sequential recurrence of Eq. 6 for any chunk size, forward and backward.  Plain
numpy, one head at a time, no blocking beyond the chunks the algorithm states.

Notation (Algorithm 1 / App. B): C chunk size; G = chunk-local inclusive
cumulative sum of log a (the paper's "A-arrow" in log space); I = 1 - a;
D_ij[s] = exp(G_i[s] - G_j[s]) for j <= i inside a chunk.

Two chunk primitives cover both passes and the whole backward:

  value_side(xq, xk, w)  -- "gsa_fwd" with GATE_K = False (pass 1): decay acts on
      the value/slot side.  out_i[s] = sum_{j<=i} <xq_i, xk_j> w_j[s] prod_{r=j+1..i} a_r[s]
      with state S (d x m).
  key_side(uq, uk, xv)   -- "gsa_fwd" with GATE_K = True (pass 2): decay acts on
      the key/slot side.   out_i = sum_{j<=i} (sum_s uq_i[s] uk_j[s] prod_{r=j+1..i} a_r[s]) xv_j
      with state S (m x d).

Each also runs time-reversed (sum over i >= j, same decay product), which is
what the gradients w.r.t. keys, values and the input gate are.
"""
from __future__ import annotations

import numpy as np


def chunk_cumsum(g, C):
    """chunk_cumsum of Algorithm 1 in log space: G[i] = sum of g over the rows of
    i's chunk up to and including i."""
    T = g.shape[0]
    G = np.empty_like(g)
    for n0 in range(0, T, C):
        G[n0:n0 + C] = np.cumsum(g[n0:n0 + C], axis=0)
    return G


def _chunks(T, C, reverse):
    starts = list(range(0, T, C))
    return reversed(starts) if reverse else starts


def value_side(xq, xk, w, G, C, S0=None, reverse=False):
    """Pass-1 primitive.  xq, xk [T,d]; w, G [T,m]; S0 [d,m] or None.
    Returns (out [T,m], S_end [d,m])."""
    T, d = xq.shape
    m = w.shape[1]
    S = np.zeros((d, m)) if S0 is None else np.array(S0, dtype=np.float64)
    out = np.zeros((T, m))
    for n0 in _chunks(T, C, reverse):
        sl = slice(n0, min(n0 + C, T))
        Q, K, W, g = xq[sl], xk[sl], w[sl], G[sl]
        gC = g[-1]
        c = Q.shape[0]
        P = Q @ K.T                                   # [c, c]
        # D[i, j, s] = exp(G_i - G_j), kept only where the exponent is <= 0
        diff = g[:, None, :] - g[None, :, :]
        if not reverse:
            mask = np.tril(np.ones((c, c), dtype=bool))
            D = np.where(mask[:, :, None], np.exp(np.where(mask[:, :, None], diff, 0.0)), 0.0)
            inter = (Q @ S) * np.exp(g)
            intra = np.einsum("ij,ijs,js->is", P, D, W)
            S = S * np.exp(gC)[None, :] + K.T @ (W * np.exp(gC - g))
        else:
            mask = np.triu(np.ones((c, c), dtype=bool))      # row j, col i >= j
            Dt = np.where(mask[:, :, None], np.exp(np.where(mask[:, :, None], -diff, 0.0)), 0.0)
            inter = (Q @ S) * np.exp(gC - g)
            intra = np.einsum("ji,jis,is->js", P, Dt, W)
            S = S * np.exp(gC)[None, :] + K.T @ (W * np.exp(g))
        out[sl] = inter + intra
    return out, S


def key_side(uq, uk, xv, G, C, S0=None, reverse=False):
    """Pass-2 primitive.  uq, uk, G [T,m]; xv [T,d]; S0 [m,d] or None.
    Returns (out [T,d], S_end [m,d])."""
    T, m = uq.shape
    d = xv.shape[1]
    S = np.zeros((m, d)) if S0 is None else np.array(S0, dtype=np.float64)
    out = np.zeros((T, d))
    for n0 in _chunks(T, C, reverse):
        sl = slice(n0, min(n0 + C, T))
        Uq, Uk, V, g = uq[sl], uk[sl], xv[sl], G[sl]
        gC = g[-1]
        c = Uq.shape[0]
        diff = g[:, None, :] - g[None, :, :]
        if not reverse:
            mask = np.tril(np.ones((c, c), dtype=bool))
            D = np.where(mask[:, :, None], np.exp(np.where(mask[:, :, None], diff, 0.0)), 0.0)
            A = np.einsum("is,js,ijs->ij", Uq, Uk, D)
            o = (Uq * np.exp(g)) @ S + A @ V
            S = np.exp(gC)[:, None] * S + (Uk * np.exp(gC - g)).T @ V
        else:
            mask = np.triu(np.ones((c, c), dtype=bool))
            Dt = np.where(mask[:, :, None], np.exp(np.where(mask[:, :, None], -diff, 0.0)), 0.0)
            A = np.einsum("js,is,jis->ji", Uq, Uk, Dt)
            o = (Uq * np.exp(gC - g)) @ S + A @ V
            S = np.exp(gC)[:, None] * S + (Uk * np.exp(g)).T @ V
        out[sl] = o
    return out, S


def _softmax(z):
    z = z - z.max(axis=-1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=-1, keepdims=True)


def gsa_fwd_chunk(q, k, v, a, C, K0=None, V0=None, scale=1.0):
    """ForwardPass of Algorithm 1 for one head (a strictly inside (0,1]).
    Returns dict(o, ok, KT, VT, p, G)."""
    g = np.log(a)
    G = chunk_cumsum(g, C)
    I = 1.0 - a
    okraw, Sk = value_side(q, k, I, G, C, None if K0 is None else np.asarray(K0).T)
    ok = scale * okraw
    p = _softmax(ok)
    o, Sv = key_side(p, I, v, G, C, V0)
    return dict(o=o, ok=ok, KT=Sk.T, VT=Sv, p=p, G=G)


def gsa_bwd_chunk(q, k, v, a, dO, C, K0=None, V0=None, dKT=None, dVT=None, scale=1.0):
    """BackwardPass of Algorithm 1 for one head, un-garbled: every gradient is a
    forward or time-reversed run of one of the two primitives, and the forget
    gate gradient is the reversed cumulative sum the paper states (App. B),
    taken over the whole sequence.  Returns dict(dq, dk, dv, da, dg, dK0, dV0)
    with da / dg the total derivative w.r.t. a / log a."""
    f = gsa_fwd_chunk(q, k, v, a, C, K0, V0, scale)
    G, p, ok = f["G"], f["p"], f["ok"]
    I = 1.0 - a
    # pass 2 backward: gradient w.r.t. its queries p
    dp, _ = value_side(dO, v, I, G, C, None if V0 is None else np.asarray(V0).T)
    # softmax backward
    dok = p * (dp - (p * dp).sum(-1, keepdims=True))
    dz = scale * dok                     # gradient w.r.t. the unscaled pass-1 output
    # pass 1 backward: gradient w.r.t. q
    dq, _ = key_side(dz, I, k, G, C, K0)
    # time-reversed runs: gradients w.r.t. v, k and the input gate I
    dv, dV0 = key_side(I, p, dO, G, C, dVT, reverse=True)
    dIv, _ = value_side(v, dO, p, G, C, None if dVT is None else np.asarray(dVT).T, reverse=True)
    dk, dK0 = key_side(I, dz, q, G, C, dKT, reverse=True)
    dIk, _ = value_side(k, q, dz, G, C, None if dKT is None else np.asarray(dKT).T, reverse=True)
    dI = dIk + dIv
    # forget-gate gradient through the decays: reversed cumulative sum
    u = p * dp + ok * dok - I * dI
    dlog = np.cumsum(u[::-1], axis=0)[::-1].copy()
    if dKT is not None:
        dlog += (np.asarray(dKT) * f["KT"]).sum(-1)[None, :]
    if dVT is not None:
        dlog += (np.asarray(dVT) * f["VT"]).sum(-1)[None, :]
    da = dlog / a - dI
    dg = dlog - a * dI
    return dict(dq=dq, dk=dk, dv=dv, da=da, dg=dg, dK0=dK0, dV0=dV0)
