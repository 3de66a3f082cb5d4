"""CPU pins for the sequential fp64 oracle (no GPU, no CUDA library).

Each test ties the oracle to something other than itself: the brute-force
unrolled form of Eq. 7, closed forms, textbook special cases computed by a
library routine, invariants of Eq. 6, finite differences and autograd.
"""
import numpy as np
import pytest
import torch
from scipy.signal import lfilter

import oracle
from oracle import chunkwise, unrolled


def rand_problem(seed, B=1, T=12, H=2, dk=5, dv=4, m=3, init=False):
    r = np.random.default_rng(seed)
    q = r.standard_normal((B, T, H, dk))
    k = r.standard_normal((B, T, H, dk))
    v = r.standard_normal((B, T, H, dv))
    a = 1.0 / (1.0 + np.exp(-r.standard_normal((B, T, H, m))))
    K0 = r.standard_normal((B, H, m, dk)) * 0.5 if init else None
    V0 = r.standard_normal((B, H, m, dv)) * 0.5 if init else None
    return q, k, v, a, K0, V0


# ---------------------------------------------------------------- forward pins
@pytest.mark.parametrize("init", [False, True])
@pytest.mark.parametrize("scale", [1.0, 0.37])
def test_fwd_matches_bruteforce_unrolled_form(init, scale):
    q, k, v, a, K0, V0 = rand_problem(1, T=17, H=2, dk=6, dv=5, m=4, init=init)
    r = oracle.fwd(q, k, v, a, K0=K0, V0=V0, scale=scale)
    for h in range(2):
        o, logits, KT, VT = unrolled.gsa_unrolled(
            q[0, :, h], k[0, :, h], v[0, :, h], a[0, :, h],
            None if K0 is None else K0[0, h], None if V0 is None else V0[0, h], scale)
        np.testing.assert_allclose(r["o"][0, :, h], o.numpy(), rtol=0, atol=1e-12)
        np.testing.assert_allclose(r["ok"][0, :, h], logits.numpy(), rtol=0, atol=1e-12)
        np.testing.assert_allclose(r["KT"][0, h], KT.numpy(), rtol=0, atol=1e-12)
        np.testing.assert_allclose(r["VT"][0, h], VT.numpy(), rtol=0, atol=1e-12)


def test_gate_zero_returns_values_for_any_initial_state():
    # a == 0: every slot row is overwritten by (k_t, v_t); the softmax is uniform
    # over m identical rows, so o_t = v_t exactly.
    q, k, v, a, K0, V0 = rand_problem(2, T=9, init=True)
    r = oracle.fwd(q, k, v, np.zeros_like(a), K0=K0, V0=V0)
    np.testing.assert_allclose(r["o"], v, rtol=0, atol=1e-14)


def test_single_slot_is_first_order_iir_filter():
    # m == 1: softmax over one slot is 1, so o_t = a o_{t-1} + (1-a) v_t,
    # independent of q and k.  Constant a makes it scipy's lfilter.
    q, k, v, _, _, _ = rand_problem(3, T=40, H=1, dk=3, dv=2, m=1)
    alpha = 0.83
    a = np.full((1, 40, 1, 1), alpha)
    r = oracle.fwd(q, k, v, a)
    ref = lfilter([1 - alpha], [1.0, -alpha], v[0, :, 0, :], axis=0)
    np.testing.assert_allclose(r["o"][0, :, 0], ref, rtol=0, atol=1e-13)


def test_gate_one_is_softmax_attention_over_fixed_slots():
    # a == 1: the memories never change, so o_t = V0^T softmax(K0 q_t), i.e.
    # ordinary (non-causal) softmax attention of q_t over m key/value rows.
    q, k, v, a, K0, V0 = rand_problem(4, T=11, H=2, dk=8, dv=6, m=5, init=True)
    scale = 8 ** -0.5
    r = oracle.fwd(q, k, v, np.ones_like(a), K0=K0, V0=V0, scale=scale)
    tq = torch.tensor(q).permute(0, 2, 1, 3)                      # [B,H,T,dk]
    ref = torch.nn.functional.scaled_dot_product_attention(
        tq, torch.tensor(K0), torch.tensor(V0), scale=scale)
    np.testing.assert_allclose(r["o"], ref.permute(0, 2, 1, 3).numpy(), rtol=0, atol=1e-13)
    np.testing.assert_allclose(r["KT"], K0, rtol=0, atol=0)
    # and with empty memories nothing is ever written
    r0 = oracle.fwd(q, k, v, np.ones_like(a))
    assert np.all(r0["o"] == 0)


def test_constant_gate_constant_kv_closed_form():
    # constant per-slot gate alpha_s and constant k, v: K~_t[s] = (1 - alpha_s^t) kbar
    T, dk, dv, m = 15, 4, 3, 5
    r = np.random.default_rng(5)
    kbar, vbar = r.standard_normal(dk), r.standard_normal(dv)
    alpha = r.uniform(0.2, 0.95, m)
    q = r.standard_normal((1, T, 1, dk))
    k = np.broadcast_to(kbar, (1, T, 1, dk)).copy()
    v = np.broadcast_to(vbar, (1, T, 1, dv)).copy()
    a = np.broadcast_to(alpha, (1, T, 1, m)).copy()
    res = oracle.fwd(q, k, v, a)
    for t in range(T):
        w = 1 - alpha ** (t + 1)
        z = w * (kbar @ q[0, t, 0])
        p = np.exp(z - z.max()); p /= p.sum()
        np.testing.assert_allclose(res["o"][0, t, 0], (p * w).sum() * vbar, rtol=0, atol=1e-13)


def test_invariants_slot_permutation_convexity_head_independence():
    q, k, v, a, K0, V0 = rand_problem(6, B=2, T=10, H=2, m=4, init=True)
    base = oracle.fwd(q, k, v, a, K0=K0, V0=V0)
    perm = np.array([2, 0, 3, 1])
    pr = oracle.fwd(q, k, v, a[..., perm], K0=K0[:, :, perm], V0=V0[:, :, perm])
    np.testing.assert_allclose(pr["o"], base["o"], rtol=0, atol=1e-13)
    np.testing.assert_allclose(pr["KT"], base["KT"][:, :, perm], rtol=0, atol=1e-14)
    # rows of V~ are convex combinations of past v: v == c, empty memory =>
    # o_t = c * sum_s p_s (1 - prod a[s])
    c = np.array([1.5, -2.0, 0.25, 3.0])
    vc = np.broadcast_to(c, v.shape).copy()
    res = oracle.fwd(q, k, vc, a)
    lo = res["ok"]
    p = np.exp(lo - lo.max(-1, keepdims=True)); p /= p.sum(-1, keepdims=True)
    fill = 1 - np.cumprod(a, axis=1)
    np.testing.assert_allclose(res["o"], (p * fill).sum(-1, keepdims=True) * c, rtol=0, atol=1e-13)
    # (b,h) pairs are independent: changing one pair's inputs leaves the others
    q2 = q.copy(); q2[1, :, 0] += 1.0
    other = oracle.fwd(q2, k, v, a, K0=K0, V0=V0)
    np.testing.assert_array_equal(other["o"][0], base["o"][0])
    np.testing.assert_array_equal(other["o"][1, :, 1], base["o"][1, :, 1])
    assert np.abs(other["o"][1, :, 0] - base["o"][1, :, 0]).max() > 1e-3


def test_state_carry_and_bh_range_and_log_gate():
    q, k, v, a, K0, V0 = rand_problem(7, B=2, T=14, H=3, init=True)
    full = oracle.fwd(q, k, v, a, K0=K0, V0=V0)
    first = oracle.fwd(q[:, :6], k[:, :6], v[:, :6], a[:, :6], K0=K0, V0=V0)
    second = oracle.fwd(q[:, 6:], k[:, 6:], v[:, 6:], a[:, 6:], K0=first["KT"], V0=first["VT"])
    np.testing.assert_allclose(np.concatenate([first["o"], second["o"]], 1), full["o"], atol=1e-14)
    np.testing.assert_allclose(second["KT"], full["KT"], atol=1e-14)
    part = oracle.fwd(q, k, v, a, K0=K0, V0=V0, bh_range=(2, 5), threads=2)
    o_flat = lambda x: x.transpose(0, 2, 1, 3).reshape(6, 14, -1)
    np.testing.assert_array_equal(o_flat(part["o"])[2:5], o_flat(full["o"])[2:5])
    assert np.all(o_flat(part["o"])[:2] == 0) and np.all(o_flat(part["o"])[5:] == 0)
    lg = oracle.fwd(q, k, v, np.log(a), gate_is_log=True, K0=K0, V0=V0)
    np.testing.assert_allclose(lg["o"], full["o"], atol=1e-13)


def test_decode_steps_reproduce_forward():
    q, k, v, a, K0, V0 = rand_problem(8, B=3, T=9, H=2, init=True)
    full = oracle.fwd(q, k, v, a, K0=K0, V0=V0, scale=0.7)
    Ks, Vs = K0.copy(), V0.copy()
    for t in range(9):
        o = oracle.decode_step(q[:, t], k[:, t], v[:, t], a[:, t], Ks, Vs, scale=0.7)
        np.testing.assert_allclose(o, full["o"][:, t], atol=1e-14)
    np.testing.assert_allclose(Ks, full["KT"], atol=1e-14)
    np.testing.assert_allclose(Vs, full["VT"], atol=1e-14)


# --------------------------------------------------------------- backward pins
def _loss_np(q, k, v, a, K0, V0, dO, dKT, dVT, scale, log):
    r = oracle.fwd(q, k, v, a, K0=K0, V0=V0, scale=scale, gate_is_log=log)
    return (r["o"] * dO).sum() + (r["KT"] * dKT).sum() + (r["VT"] * dVT).sum()


@pytest.mark.parametrize("log", [False, True])
def test_bwd_matches_central_finite_differences(log):
    q, k, v, a, K0, V0 = rand_problem(9, B=1, T=7, H=2, dk=4, dv=3, m=3, init=True)
    gate = np.log(a) if log else a
    r = np.random.default_rng(10)
    dO = r.standard_normal(v.shape)
    dKT = r.standard_normal(K0.shape); dVT = r.standard_normal(V0.shape)
    scale = 0.8
    g = oracle.bwd(q, k, v, gate, dO, K0=K0, V0=V0, dKT=dKT, dVT=dVT, scale=scale, gate_is_log=log)
    args = dict(q=q, k=k, v=v, a=gate, K0=K0, V0=V0)
    names = dict(q="dq", k="dk", v="dv", a="dgate", K0="dK0", V0="dV0")
    eps = 1e-6
    for nm, gn in names.items():
        x = args[nm]
        idx = [tuple(r.integers(0, s) for s in x.shape) for _ in range(12)]
        for ix in idx:
            xp = {kk: vv.copy() for kk, vv in args.items()}
            xm = {kk: vv.copy() for kk, vv in args.items()}
            xp[nm][ix] += eps; xm[nm][ix] -= eps
            fd = (_loss_np(**xp, dO=dO, dKT=dKT, dVT=dVT, scale=scale, log=log)
                  - _loss_np(**xm, dO=dO, dKT=dKT, dVT=dVT, scale=scale, log=log)) / (2 * eps)
            assert abs(fd - g[gn][ix]) < 1e-7 * max(1.0, abs(fd)), (nm, ix, fd, g[gn][ix])


def test_bwd_matches_autograd_of_unrolled_form():
    q, k, v, a, K0, V0 = rand_problem(11, B=1, T=10, H=1, dk=5, dv=4, m=3, init=True)
    r = np.random.default_rng(12)
    dO = r.standard_normal(v.shape)
    dKT = r.standard_normal(K0.shape); dVT = r.standard_normal(V0.shape)
    g = oracle.bwd(q, k, v, a, dO, K0=K0, V0=V0, dKT=dKT, dVT=dVT, scale=1.3)
    ts = [torch.tensor(x[0, :, 0] if x.ndim == 4 and x.shape[1] == 10 else x[0, 0],
                       requires_grad=True) for x in (q, k, v, a, K0, V0)]
    o, _, KT, VT = unrolled.gsa_unrolled(*ts, scale=1.3)
    loss = (o * torch.tensor(dO[0, :, 0])).sum() + (KT * torch.tensor(dKT[0, 0])).sum() \
        + (VT * torch.tensor(dVT[0, 0])).sum()
    grads = torch.autograd.grad(loss, ts)
    for name, gt, sel in zip(("dq", "dk", "dv", "dgate", "dK0", "dV0"), grads,
                             (0, 0, 0, 0, 1, 1)):
        mine = g[name][0, :, 0] if sel == 0 else g[name][0, 0]
        np.testing.assert_allclose(mine, gt.numpy(), rtol=0, atol=1e-11, err_msg=name)


def test_bwd_special_cases():
    q, k, v, a, K0, V0 = rand_problem(13, T=8, init=True)
    dO = np.random.default_rng(14).standard_normal(v.shape)
    # a == 0 => o = v: dv = dO, nothing flows to q, k or the initial memories
    g = oracle.bwd(q, k, v, np.zeros_like(a), dO, K0=K0, V0=V0)
    np.testing.assert_allclose(g["dv"], dO, atol=1e-14)
    for nm in ("dq", "dk", "dK0", "dV0"):
        assert np.abs(g[nm]).max() < 1e-13, nm
    # linear in dO
    g1 = oracle.bwd(q, k, v, a, dO, K0=K0, V0=V0)
    g2 = oracle.bwd(q, k, v, a, -2.5 * dO, K0=K0, V0=V0)
    for nm in ("dq", "dk", "dv", "dgate", "dK0", "dV0"):
        np.testing.assert_allclose(g2[nm], -2.5 * g1[nm], atol=1e-12)


# ---------------------------------------- chunkwise regrouping == step by step
@pytest.mark.parametrize("C", [16, 32, 64])
@pytest.mark.parametrize("T", [64, 100])
def test_chunkwise_forward_equals_stepwise(C, T):
    q, k, v, a, K0, V0 = rand_problem(15, B=1, T=T, H=1, dk=8, dv=6, m=5, init=True)
    a = a ** 0.25
    seq = oracle.fwd(q, k, v, a, K0=K0, V0=V0, scale=0.9)
    ch = chunkwise.gsa_fwd_chunk(q[0, :, 0], k[0, :, 0], v[0, :, 0], a[0, :, 0], C,
                                 K0[0, 0], V0[0, 0], 0.9)
    np.testing.assert_allclose(ch["o"], seq["o"][0, :, 0], atol=1e-12)
    np.testing.assert_allclose(ch["ok"], seq["ok"][0, :, 0], atol=1e-12)
    np.testing.assert_allclose(ch["KT"], seq["KT"][0, 0], atol=1e-12)
    np.testing.assert_allclose(ch["VT"], seq["VT"][0, 0], atol=1e-12)


def test_chunkwise_strong_forgetting_stays_finite():
    # gates near 0 make the naive ratio form overflow; the masked-exponent form must not
    q, k, v, a, _, _ = rand_problem(16, B=1, T=128, H=1, dk=4, dv=4, m=3)
    a = 1.0 / (1.0 + np.exp(6.0 + 2 * np.random.default_rng(17).standard_normal(a.shape)))
    seq = oracle.fwd(q, k, v, a)
    ch = chunkwise.gsa_fwd_chunk(q[0, :, 0], k[0, :, 0], v[0, :, 0], a[0, :, 0], 64)
    assert np.isfinite(ch["o"]).all()
    np.testing.assert_allclose(ch["o"], seq["o"][0, :, 0], atol=1e-12)


@pytest.mark.parametrize("C", [16, 64])
@pytest.mark.parametrize("with_final", [False, True])
def test_chunkwise_backward_and_gate_identity_equal_sweep(C, with_final):
    T = 80
    q, k, v, a, K0, V0 = rand_problem(18, B=1, T=T, H=1, dk=6, dv=5, m=4, init=True)
    a = a ** 0.25
    r = np.random.default_rng(19)
    dO = r.standard_normal(v.shape)
    dKT = r.standard_normal(K0.shape) if with_final else None
    dVT = r.standard_normal(V0.shape) if with_final else None
    g = oracle.bwd(q, k, v, a, dO, K0=K0, V0=V0, dKT=dKT, dVT=dVT, scale=1.1)
    glog = oracle.bwd(q, k, v, np.log(a), dO, K0=K0, V0=V0, dKT=dKT, dVT=dVT, scale=1.1,
                      gate_is_log=True)
    ch = chunkwise.gsa_bwd_chunk(q[0, :, 0], k[0, :, 0], v[0, :, 0], a[0, :, 0], dO[0, :, 0], C,
                                 K0[0, 0], V0[0, 0],
                                 None if dKT is None else dKT[0, 0],
                                 None if dVT is None else dVT[0, 0], 1.1)
    np.testing.assert_allclose(ch["dq"], g["dq"][0, :, 0], atol=1e-11)
    np.testing.assert_allclose(ch["dk"], g["dk"][0, :, 0], atol=1e-11)
    np.testing.assert_allclose(ch["dv"], g["dv"][0, :, 0], atol=1e-11)
    np.testing.assert_allclose(ch["da"], g["dgate"][0, :, 0], atol=1e-10)
    np.testing.assert_allclose(ch["dg"], glog["dgate"][0, :, 0], atol=1e-10)
    np.testing.assert_allclose(ch["dK0"], g["dK0"][0, 0], atol=1e-11)
    np.testing.assert_allclose(ch["dV0"], g["dV0"][0, 0], atol=1e-11)


# ------------------------------------------------------------------ gate from logits (Sec. 3.3)
def test_logit_gate_equals_explicit_damped_sigmoid_and_chain_rule():
    # a = sigmoid(x)^(1/tau): the logits mode must equal the linear-gate mode fed with that a, and
    # its gate gradient the linear one times da/dx; tau = 1 is the plain sigmoid
    r = np.random.default_rng(11)
    B, T, H, d, m = 2, 9, 2, 4, 3
    q, k, v, dO = (r.standard_normal((B, T, H, d)) for _ in range(4))
    x = 2.0 * r.standard_normal((B, T, H, m))
    for tau in (1.0, 8.0):
        sig = 1.0 / (1.0 + np.exp(-x))
        a = sig ** (1.0 / tau)
        f_log, f_lin = oracle.fwd(q, k, v, x, gate_is_logits=True, tau=tau), oracle.fwd(q, k, v, a)
        for n in ("o", "ok", "KT", "VT"):
            assert np.abs(f_log[n] - f_lin[n]).max() < 1e-13
        b_log = oracle.bwd(q, k, v, x, dO, gate_is_logits=True, tau=tau)
        b_lin = oracle.bwd(q, k, v, a, dO)
        for n in ("dq", "dk", "dv"):
            assert np.abs(b_log[n] - b_lin[n]).max() < 1e-13
        assert np.abs(b_log["dgate"] - b_lin["dgate"] * a * (1 - sig) / tau).max() < 1e-12


def test_logit_gate_gradient_matches_central_finite_differences():
    r = np.random.default_rng(12)
    B, T, H, d, m = 1, 7, 1, 3, 2
    q, k, v, dO = (r.standard_normal((B, T, H, d)) for _ in range(4))
    x = r.standard_normal((B, T, H, m))
    f = lambda x_: float((oracle.fwd(q, k, v, x_, gate_is_logits=True, tau=8.0)["o"] * dO).sum())
    g = oracle.bwd(q, k, v, x, dO, gate_is_logits=True, tau=8.0)["dgate"]
    eps = 1e-6
    for idx in np.ndindex(*x.shape):
        xp, xm = x.copy(), x.copy()
        xp[idx] += eps
        xm[idx] -= eps
        assert abs((f(xp) - f(xm)) / (2 * eps) - g[idx]) < 1e-7


def test_logit_gate_decode_steps_reproduce_forward():
    r = np.random.default_rng(13)
    S, T, H, d, m = 2, 5, 2, 4, 3
    q, k, v = (r.standard_normal((S, T, H, d)) for _ in range(3))
    x = r.standard_normal((S, T, H, m))
    ref = oracle.fwd(q, k, v, x, gate_is_logits=True, tau=8.0)
    Ks, Vs = np.zeros((S, H, m, d)), np.zeros((S, H, m, d))
    for t in range(T):
        o = oracle.decode_step(q[:, t], k[:, t], v[:, t], x[:, t], Ks, Vs, gate_is_logits=True, tau=8.0)
        assert np.abs(o - ref["o"][:, t]).max() < 1e-13
    assert np.abs(Ks - ref["KT"]).max() < 1e-13


# ------------------------------------- the ablation's replacements of the slot softmax
ACTS = ["none", "relu", "swish", "relu2"]


@pytest.mark.parametrize("act", ACTS)
def test_slot_activation_variants_match_unrolled_form_and_its_autograd(act):
    """Forward against the unrolled two-pass form with the library's activation routine, every
    gradient against autograd of that form (the paper's ablation on the non-linearity)."""
    T = 10
    q, k, v, a, K0, V0 = rand_problem(31, B=1, T=T, H=1, dk=5, dv=4, m=3, init=True)
    r = np.random.default_rng(32)
    dO = r.standard_normal(v.shape)
    dKT = r.standard_normal(K0.shape); dVT = r.standard_normal(V0.shape)
    f = oracle.fwd(q, k, v, a, K0=K0, V0=V0, scale=0.9, act=act)
    g = oracle.bwd(q, k, v, a, dO, K0=K0, V0=V0, dKT=dKT, dVT=dVT, scale=0.9, act=act)
    ts = [torch.tensor(x[0, :, 0] if x.ndim == 4 and x.shape[1] == T else x[0, 0],
                       requires_grad=True) for x in (q, k, v, a, K0, V0)]
    o, logits, KT, VT = unrolled.gsa_unrolled(*ts, scale=0.9, act=act)
    np.testing.assert_allclose(f["o"][0, :, 0], o.detach().numpy(), rtol=0, atol=1e-12)
    np.testing.assert_allclose(f["ok"][0, :, 0], logits.detach().numpy(), rtol=0, atol=1e-12)
    if act in ("relu", "relu2"):      # both signs occur, so the kink is exercised on either side
        assert (logits.detach().numpy() > 0).any() and (logits.detach().numpy() < 0).any()
    loss = (o * torch.tensor(dO[0, :, 0])).sum() + (KT * torch.tensor(dKT[0, 0])).sum() \
        + (VT * torch.tensor(dVT[0, 0])).sum()
    grads = torch.autograd.grad(loss, ts)
    for name, gt, sel in zip(("dq", "dk", "dv", "dgate", "dK0", "dV0"), grads, (0, 0, 0, 0, 1, 1)):
        mine = g[name][0, :, 0] if sel == 0 else g[name][0, 0]
        np.testing.assert_allclose(mine, gt.numpy(), rtol=0, atol=1e-11, err_msg=name)


def test_slot_activation_none_is_a_double_sum_without_memories():
    """Without a non-linearity the layer is bilinear in the two passes:
    o_t = scale * sum_{i,j<=t} (sum_s W[t,i,s] W[t,j,s]) <q_t, k_j> v_i."""
    T, m = 9, 3
    q, k, v, a, _, _ = rand_problem(33, B=1, T=T, H=1, dk=4, dv=3, m=m)
    f = oracle.fwd(q, k, v, a, scale=0.6, act="none")
    qq, kk, vv, aa = q[0, :, 0], k[0, :, 0], v[0, :, 0], a[0, :, 0]
    for t in range(T):
        W = np.zeros((t + 1, m))
        for j in range(t + 1):
            W[j] = (1 - aa[j]) * np.prod(aa[j + 1:t + 1], axis=0)
        o = np.zeros(3)
        for i in range(t + 1):
            for j in range(t + 1):
                o += 0.6 * (W[i] * W[j]).sum() * (qq[t] @ kk[j]) * vv[i]
        np.testing.assert_allclose(f["o"][0, t, 0], o, rtol=0, atol=1e-12)


def test_slot_activation_relations_and_decode():
    """ReLU on all-positive logits is the identity; squared ReLU is ReLU with the logits as
    weights once more; decode steps reproduce the forward for a replacement too."""
    q, k, v, a, K0, V0 = rand_problem(34, B=2, T=8, H=2, init=True)
    q, k, K0p = np.abs(q), np.abs(k), np.abs(K0)
    none = oracle.fwd(q, k, v, a, K0=K0p, V0=V0, scale=0.5, act="none")
    relu = oracle.fwd(q, k, v, a, K0=K0p, V0=V0, scale=0.5, act="relu")
    assert (none["ok"] > 0).all()
    np.testing.assert_allclose(relu["o"], none["o"], rtol=0, atol=1e-14)
    full = oracle.fwd(q, k, v, a, K0=K0, V0=V0, scale=0.7, act="swish")
    Ks, Vs = K0.copy(), V0.copy()
    for t in range(8):
        o = oracle.decode_step(q[:, t], k[:, t], v[:, t], a[:, t], Ks, Vs, scale=0.7, act="swish")
        np.testing.assert_allclose(o, full["o"][:, t], atol=1e-14)
    np.testing.assert_allclose(Ks, full["KT"], atol=1e-14)


# ---------------------------------------------------------------- packed sequences
def test_packed_sequences_match_the_unrolled_form_of_every_sequence_and_finite_differences():
    """fwd_packed / bwd_packed (variable-length sequences back to back along T, memories emptied at
    every offset): each sequence against the brute-force unrolled form on its own slice, and the
    assembled gradients (which sequence receives K0 / dKT) against central finite differences."""
    q, k, v, a, K0, V0 = rand_problem(31, T=19, H=2, dk=4, dv=3, m=3, init=True)
    cu = [0, 5, 6, 14, 19]
    r = oracle.fwd_packed(q, k, v, a, cu, K0=K0, V0=V0, scale=0.7)
    for i in range(len(cu) - 1):
        sl = slice(cu[i], cu[i + 1])
        for h in range(2):
            o, logits, KT, VT = unrolled.gsa_unrolled(q[0, sl, h], k[0, sl, h], v[0, sl, h], a[0, sl, h],
                                                      K0[0, h] if i == 0 else None, V0[0, h] if i == 0 else None, 0.7)
            np.testing.assert_allclose(r["o"][0, sl, h], o.numpy(), rtol=1e-10, atol=1e-12)
            np.testing.assert_allclose(r["ok"][0, sl, h], logits.numpy(), rtol=1e-10, atol=1e-12)
            if i == len(cu) - 2:
                np.testing.assert_allclose(r["KT"][0, h], KT.numpy(), rtol=1e-10, atol=1e-12)
    rng = np.random.default_rng(5)
    dO = rng.standard_normal(v.shape)
    dKT, dVT = rng.standard_normal(K0.shape), rng.standard_normal(V0.shape)

    def loss(q_, k_, v_, a_, K0_, V0_):
        f = oracle.fwd_packed(q_, k_, v_, a_, cu, K0=K0_, V0=V0_, scale=0.7)
        return float((f["o"] * dO).sum() + (f["KT"] * dKT).sum() + (f["VT"] * dVT).sum())

    g = oracle.bwd_packed(q, k, v, a, dO, cu, K0=K0, V0=V0, dKT=dKT, dVT=dVT, scale=0.7)
    args = [q, k, v, a, K0, V0]
    eps = 1e-6
    for pos, name in ((0, "dq"), (1, "dk"), (2, "dv"), (3, "dgate"), (4, "dK0"), (5, "dV0")):
        x = args[pos]
        for _ in range(6):
            idx = tuple(rng.integers(0, n) for n in x.shape)
            hi, lo = [t.copy() for t in args], [t.copy() for t in args]
            hi[pos][idx] += eps
            lo[pos][idx] -= eps
            fd = (loss(*hi) - loss(*lo)) / (2 * eps)
            assert abs(fd - g[name][idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx, fd, g[name][idx])


# ---------------------------------------------------------------- layer pre- and post-operations
def test_layer_elementwise_ops_against_library_routines_closed_form_and_autograd():
    """Swish (feature map of q, k, v) and Swish -> RMSNorm (output path): against torch's silu and
    rms_norm in fp64, a closed form on constant rows, autograd, and central finite differences."""
    from oracle import layer
    r = np.random.default_rng(12)
    x = r.standard_normal((2, 5, 3, 8)) * 2.0
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    np.testing.assert_allclose(layer.swish(x), torch.nn.functional.silu(xt).detach().numpy(), rtol=1e-13, atol=1e-15)
    torch.nn.functional.silu(xt).sum().backward()
    np.testing.assert_allclose(layer.swish_grad(x), xt.grad.numpy(), rtol=1e-12, atol=1e-14)

    w = r.standard_normal(24) * 0.5 + 1.0
    eps = 1e-5
    y = layer.out_norm_fwd(x, w, eps)
    ot = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    wt = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    yt = torch.nn.functional.rms_norm(torch.nn.functional.silu(ot).reshape(2, 5, 24), (24,), wt, eps).reshape(2, 5, 3, 8)
    np.testing.assert_allclose(y, yt.detach().numpy(), rtol=1e-12, atol=1e-14)
    dy = r.standard_normal(x.shape)
    (yt * torch.tensor(dy)).sum().backward()
    do, dw = layer.out_norm_bwd(x, dy, w, eps)
    np.testing.assert_allclose(do, ot.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(dw, wt.grad.numpy(), rtol=1e-10, atol=1e-12)
    # constant rows: every value of a token equal to c  ->  Swish(c) / sqrt(Swish(c)^2 + eps)
    c = 1.7
    sc = c / (1 + np.exp(-c))
    yc = layer.out_norm_fwd(np.full((1, 2, 3, 8), c), None, eps)
    np.testing.assert_allclose(yc, sc / np.sqrt(sc * sc + eps), rtol=1e-13)
    # finite differences of a scalar loss through the forward
    h = 1e-6
    for _ in range(6):
        idx = tuple(r.integers(0, n) for n in x.shape)
        hi, lo = x.copy(), x.copy()
        hi[idx] += h
        lo[idx] -= h
        fd = ((layer.out_norm_fwd(hi, w, eps) - layer.out_norm_fwd(lo, w, eps)) * dy).sum() / (2 * h)
        assert abs(fd - do[idx]) <= 1e-6 * max(1.0, abs(fd))


# ---------------------------------------------------------------- ABC (no decay) and constant decay
def test_abc_oracle_against_its_linear_attention_form_and_uniform_scores():
    """oracle/abc.py (Eq. 3-4): (i) with the cumulative softmax written out, o' = sum_{j<=t} (q_t . k_j) phi_j
    is plain causal linear attention (Eq. 5's parallel form), evaluated here with a masked matrix
    product; (ii) equal scores give phi_t = 1 / t, so the memories are running sums of k_t / t."""
    from oracle import abc
    r = np.random.default_rng(3)
    B, T, H, dk, dv, m = 1, 9, 2, 4, 3, 5
    q, k, v = r.standard_normal((B, T, H, dk)), r.standard_normal((B, T, H, dk)), r.standard_normal((B, T, H, dv))
    s = r.standard_normal((B, T, H, m))
    f = abc.fwd(q, k, v, s, scale=0.8)
    e = np.exp(s)
    phi = e / np.cumsum(e, axis=1)
    mask = np.tril(np.ones((T, T)))
    for h in range(H):
        P = (q[0, :, h] @ k[0, :, h].T) * mask                    # [T,T]
        logits = 0.8 * P @ phi[0, :, h]                            # [T,m]
        np.testing.assert_allclose(f["ok"][0, :, h], logits, rtol=1e-12, atol=1e-13)
        p = np.exp(logits - logits.max(-1, keepdims=True)); p /= p.sum(-1, keepdims=True)
        A = (p @ phi[0, :, h].T) * mask                            # [T,T]
        np.testing.assert_allclose(f["o"][0, :, h], A @ v[0, :, h], rtol=1e-12, atol=1e-13)
    f1 = abc.fwd(q, k, v, np.zeros_like(s))
    want = np.cumsum(k[0, :, 0] / np.arange(1, T + 1)[:, None], axis=0)[-1]
    np.testing.assert_allclose(f1["KT"][0, 0, 2], want, rtol=1e-12)
    # the gradients come from autograd of the definition; spot-check them with finite differences
    dO = r.standard_normal(v.shape)
    g = abc.bwd(q, k, v, s, dO, scale=0.8)
    h_ = 1e-6
    for name, x in (("dgate", s), ("dk", k)):
        for _ in range(4):
            idx = tuple(r.integers(0, n) for n in x.shape)
            hi, lo = x.copy(), x.copy()
            hi[idx] += h_; lo[idx] -= h_
            a_hi = [q, k, v, s]; a_lo = [q, k, v, s]
            pos = 3 if name == "dgate" else 1
            a_hi[pos], a_lo[pos] = hi, lo
            fd = ((abc.fwd(*a_hi, scale=0.8)["o"] - abc.fwd(*a_lo, scale=0.8)["o"]) * dO).sum() / (2 * h_)
            assert abs(fd - g[name][idx]) <= 1e-6 * max(1.0, abs(fd))
