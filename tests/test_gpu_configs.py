"""GPU parity at the full size of the five benchmark configurations, in the launch
configuration bench.py times.  The GPU runs the whole workload; the fp64 oracle is run on
sampled (batch, head) pairs (each pair is an independent recurrence, so a sample of pairs is
a sample of complete outputs) and compared element by element on those."""
import json
import os

import numpy as np
import pytest
import torch

import gsa_workloads as W
import oracle
import paper_2409_07146_b200 as gsa
from util import TC_CONFIG_BOUNDS, TC_RTOL, TOL, mixed_err, rel_err, to_dev, to_np

pytestmark = pytest.mark.gpu

REPORT = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "gpurun_out",
                      "config_parity.json")


def record(name, errs):
    try:
        os.makedirs(os.path.dirname(REPORT), exist_ok=True)
        data = json.load(open(REPORT)) if os.path.exists(REPORT) else {}
        data[name] = errs
        json.dump(data, open(REPORT, "w"), indent=1)
    except OSError:
        pass


def pair_slices(x, pairs, H):
    """Stack the [T, D] slices of the sampled (b, h) pairs as a [len(pairs), T, 1, D] batch."""
    return np.stack([x[p // H, :, p % H] for p in pairs])[:, :, None, :]


def state_slices(x, pairs, H):
    return np.stack([x[p // H, p % H] for p in pairs])[:, None]


def sample_pairs(w, n=3):
    total = w.B * w.H
    return sorted({0, total // 2 + 1 if total > 2 else total - 1, total - 1})[:n]


def run_training_config(name, with_bwd, tc_operands="paired"):
    w = W.CONFIGS[name]
    x = W.make_inputs(w)
    p = gsa.Params(w.B, w.T, w.H, w.d_k, w.d_v, w.m, io=w.io, tc_operands=tc_operands)
    q, k, v = (to_dev(x[n], w.io) for n in ("q", "k", "v"))
    gate = to_dev(x["gate"])
    K0, V0 = to_dev(x.get("K0")), to_dev(x.get("V0"))
    ok = torch.empty(w.B, w.T, w.H, w.m, device="cuda")
    KT = torch.empty(w.B, w.H, w.m, w.d_k, device="cuda")
    VT = torch.empty(w.B, w.H, w.m, w.d_v, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = gsa.gsa_fwd(p, q, k, v, gate, K0, V0, ok_save=ok, KT=KT, VT=VT, dev_status=status)
    got = dict(o=o, ok=ok, KT=KT, VT=VT)
    if with_bwd:
        dO = to_dev(x["dO"], w.io)
        dq, dk, dv, dg = gsa.gsa_bwd(p, q, k, v, gate, dO, K0, V0, ok_saved=ok, dev_status=status)
        got.update(dq=dq, dk=dk, dv=dv, dgate=dg)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "a bounded device-side wait expired"

    pairs = sample_pairs(w)
    sub = {n: pair_slices(x[n], pairs, w.H) for n in ("q", "k", "v", "gate")}
    if "K0" in x:
        sub["K0"], sub["V0"] = state_slices(x["K0"], pairs, w.H), state_slices(x["V0"], pairs, w.H)
    ref = oracle.fwd(sub["q"], sub["k"], sub["v"], sub["gate"], K0=sub.get("K0"), V0=sub.get("V0"))
    if with_bwd:
        sub["dO"] = pair_slices(x["dO"], pairs, w.H)
        ref.update(oracle.bwd(sub["q"], sub["k"], sub["v"], sub["gate"], sub["dO"], K0=sub.get("K0"),
                              V0=sub.get("V0")))
    errs = {}
    for n, t in got.items():
        g = to_np(t)
        gs = state_slices(g, pairs, w.H) if n in ("KT", "VT") else pair_slices(g, pairs, w.H)
        assert np.isfinite(gs).all(), n
        kind, rtol, limit = TC_CONFIG_BOUNDS[n]
        bound = rel_err(gs, ref[n], True) if kind == "bf16out" else mixed_err(gs, ref[n], rtol)
        errs[n] = dict(bound=bound, plain=rel_err(gs, ref[n]), limit=limit,
                       after_output_half_ulp=rel_err(gs, ref[n], True),
                       max_over_rms=float(np.abs(ref[n]).max() / np.sqrt(np.mean(ref[n] ** 2))))
    record(name if tc_operands == "paired" else name + "/" + tc_operands, dict(pairs=pairs, errors=errs))
    print(name, tc_operands, {n: (round(e["plain"], 4), round(e["bound"], 4)) for n, e in errs.items()})
    bad = {}
    for n, e in errs.items():
        if e["bound"] > e["limit"]:
            bad[n] = e
    assert not bad, bad


def test_config_train_1p3b_fwd_bwd():
    run_training_config("train_1p3b", with_bwd=True)


def test_config_t2r_7b_fwd_bwd():
    run_training_config("t2r_7b", with_bwd=True)


@pytest.mark.parametrize("regime", ["long_keep", "long_forget"])
def test_config_long_context_forward_with_carried_state(regime):
    run_training_config(regime, with_bwd=False)


def test_config_decode_1024_steps():
    w = W.CONFIGS["decode"]
    st = W.make_decode_states(w)
    Ks, Vs = to_dev(st["K"]), to_dev(st["V"])
    seqs = [0, 101, 255]                                   # sampled sequences, all heads
    Kr = np.ascontiguousarray(st["K"][seqs].astype(np.float64))
    Vr = np.ascontiguousarray(st["V"][seqs].astype(np.float64))
    p = gsa.Params(w.B, 1, w.H, w.d_k, w.d_v, w.m, io="bf16")
    worst = 0.0
    for step in range(w.T):
        x = W.make_decode_step_inputs(w, step)
        o = gsa.gsa_decode_step(p, to_dev(x["q"], "bf16"), to_dev(x["k"], "bf16"), to_dev(x["v"], "bf16"),
                                to_dev(x["gate"]), Ks, Vs)
        ro = oracle.decode_step(x["q"][seqs], x["k"][seqs], x["v"][seqs], x["gate"][seqs], Kr, Vr)
        if step % 64 == 0 or step == w.T - 1:
            worst = max(worst, rel_err(to_np(o)[seqs], ro, stored_bf16=True))
    ek, ev = rel_err(to_np(Ks)[seqs], Kr), rel_err(to_np(Vs)[seqs], Vr)
    record("decode", dict(sequences=seqs, o=worst, Kstate=ek, Vstate=ev))
    print("decode", worst, ek, ev)
    assert worst <= TOL["bf16"] and ek <= 1e-4 and ev <= 1e-4
