"""The element-wise pre- and post-operations of the layer (Sec. 3.3) on the GPU against the numpy
oracle: the Swish feature map on q, k, v inside gsa_fwd / gsa_bwd / gsa_decode_step, and the
output path Swish -> RMSNorm over the heads of a token, forward and backward."""
import numpy as np
import pytest
import torch

import gsa_workloads as W
import oracle
from oracle import layer
import paper_2409_07146_b200 as gsa
from util import BF16_IO, TOL, bf16_half_ulp, rand_inputs, rel_err, to_dev, to_np

pytestmark = pytest.mark.gpu


def activated(x, io):
    a = layer.swish(x).astype(np.float32)
    return W.round_to_bf16(a) if io == "bf16" else a


@pytest.mark.parametrize("io,impl,d,m", [("f32", "auto", 64, 32), ("bf16", "tc", 128, 64), ("bf16", "tc", 512, 64)])
def test_feature_map_fwd_bwd(io, impl, d, m):
    B, T, H = 2, 260, 2
    x = rand_inputs(17 + d, B, T, H, d, d, m, io, init=True)
    for n in ("q", "k", "v"):                      # pre-activations of a wider range than N(0,1) q
        x[n] = (x[n] * (4.0 if n == "q" else 1.5)).astype(np.float32)
        if io == "bf16":
            x[n] = W.round_to_bf16(x[n])
    p = gsa.Params(B, T, H, d, d, m, io=io, impl=impl, feature_map="swish", scale=d ** -0.5)
    q, k, v, dO = (to_dev(x[n], io) for n in ("q", "k", "v", "dO"))
    gate, K0, V0 = to_dev(x["gate"]), to_dev(x["K0"]), to_dev(x["V0"])
    ok = torch.empty(B, T, H, m, device="cuda")
    o = gsa.gsa_fwd(p, q, k, v, gate, K0, V0, ok_save=ok)
    dq, dk, dv, dg = gsa.gsa_bwd(p, q, k, v, gate, dO, K0, V0, ok_saved=ok)
    torch.cuda.synchronize()
    qa, ka, va = (activated(x[n], io) for n in ("q", "k", "v"))
    rf = oracle.fwd(qa, ka, va, x["gate"], K0=x["K0"], V0=x["V0"], scale=d ** -0.5)
    rb = oracle.bwd(qa, ka, va, x["gate"], x["dO"], K0=x["K0"], V0=x["V0"], scale=d ** -0.5)
    ref = dict(o=rf["o"], ok=rf["ok"], dgate=rb["dgate"])
    for n in ("q", "k", "v"):
        ref["d" + n] = rb["d" + n] * layer.swish_grad(x[n])
    got = dict(o=to_np(o), ok=to_np(ok), dq=to_np(dq), dk=to_np(dk), dv=to_np(dv), dgate=to_np(dg))
    errs = {n: rel_err(got[n], ref[n], io == "bf16" and n in BF16_IO) for n in got}
    if io == "bf16":
        # dq, dk, dv are rounded to bfloat16 twice here: by the scan that writes the gradient w.r.t. the
        # activated tensor, and again after the multiplication by Swish' (in place, bfloat16 storage): two
        # half-ulps of the output format are taken off instead of one
        for n in ("dq", "dk", "dv"):
            diff = np.maximum(np.abs(got[n] - ref[n]) - 2.0 * bf16_half_ulp(ref[n]), 0.0)
            errs[n] = float(diff.max() / np.sqrt(np.mean(ref[n] ** 2)))
    print("feature map", io, d, {n: float("%.2g" % e) for n, e in errs.items()})
    assert all(e <= TOL[io] for e in errs.values()), errs


def test_feature_map_in_the_decode_step():
    S, H, d, m = 3, 4, 128, 64
    w = W.CONFIGS["decode"].scaled(B=S, H=H, d_k=d, d_v=d, m=m)
    st = W.make_decode_states(w)
    Ks, Vs = to_dev(st["K"]), to_dev(st["V"])
    Kr, Vr = st["K"].astype(np.float64), st["V"].astype(np.float64)
    p = gsa.Params(S, 1, H, d, d, m, io="bf16", feature_map="swish")
    for step in range(3):
        x = W.make_decode_step_inputs(w, step)
        o = gsa.gsa_decode_step(p, to_dev(x["q"], "bf16"), to_dev(x["k"], "bf16"), to_dev(x["v"], "bf16"),
                                to_dev(x["gate"]), Ks, Vs)
        ro = oracle.decode_step(layer.swish(x["q"]), layer.swish(x["k"]), layer.swish(x["v"]), x["gate"], Kr, Vr)
    assert rel_err(to_np(o), ro, True) <= TOL["bf16"] and rel_err(to_np(Ks), Kr) <= 1e-5 and rel_err(to_np(Vs), Vr) <= 1e-5


@pytest.mark.parametrize("io,H,dv,T", [("f32", 2, 64, 37), ("bf16", 4, 512, 100), ("bf16", 5, 512, 33), ("bf16", 32, 128, 20)])
@pytest.mark.parametrize("with_weight", [False, True])
def test_output_norm_fwd_bwd(io, H, dv, T, with_weight):
    B = 2
    r = np.random.default_rng(H + dv)
    o = (1.5 * r.standard_normal((B, T, H, dv))).astype(np.float32)
    dy = r.standard_normal((B, T, H, dv)).astype(np.float32)
    if io == "bf16":
        o, dy = W.round_to_bf16(o), W.round_to_bf16(dy)
    wgt = (1.0 + 0.3 * r.standard_normal(H * dv)).astype(np.float32) if with_weight else None
    eps = 1e-5
    p = gsa.Params(B, T, H, 128, dv, 64, io=io)
    od, dyd = to_dev(o, io), to_dev(dy, io)
    wd = to_dev(wgt) if with_weight else None
    y = gsa.gsa_out_norm_fwd(p, od, wd, eps)
    d_o, dw = gsa.gsa_out_norm_bwd(p, od, dyd, wd, eps)
    torch.cuda.synchronize()
    ry = layer.out_norm_fwd(o, wgt, eps)
    rdo, rdw = layer.out_norm_bwd(o, dy, wgt, eps)
    tol = TOL[io]
    assert rel_err(to_np(y), ry, io == "bf16") <= tol
    assert rel_err(to_np(d_o), rdo, io == "bf16") <= tol
    assert rel_err(to_np(dw), rdw) <= (1e-4 if io == "f32" else 2e-3)      # fp32 sums of bf16-exact inputs
    # deterministic
    d2, dw2 = gsa.gsa_out_norm_bwd(p, od, dyd, wd, eps)
    torch.cuda.synchronize()
    assert torch.equal(d_o, d2) and torch.equal(dw, dw2)
