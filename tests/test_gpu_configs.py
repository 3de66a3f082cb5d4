"""GPU parity at the full size of the five benchmark configurations.  The GPU runs the whole
workload; the fp64 oracle is run on sampled (batch, head) pairs (each pair is an independent
recurrence, so a sample of pairs is a sample of complete outputs) and compared element by
element on those.  The training configurations run twice: as the plain gsa_fwd + gsa_bwd pair,
and exactly as bench.py times a step -- gsa_fwd_save_gate + gsa_bwd_saved_gate captured into a
CUDA graph and replayed."""
import json
import os

import numpy as np
import pytest
import torch

import gsa_workloads as W
import oracle
import paper_2409_07146_b200 as gsa
from util import BF16_IO, TC_CONFIG_BOUNDS, TC_PLAIN_CEILING, TOL, bf16_storage_check, rel_err, to_dev, to_np

pytestmark = pytest.mark.gpu

# optional JSON report of every figure the assertions look at (path given by the environment)
REPORT = os.environ.get("GSA_PARITY_REPORT")


def record(name, errs):
    if not REPORT:
        return
    try:
        os.makedirs(os.path.dirname(os.path.abspath(REPORT)), exist_ok=True)
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


def run_training_config(name, with_bwd, tc_operands="paired", launch="plain"):
    """launch = "plain": gsa_fwd + gsa_bwd as library calls.  launch = "bench": the step of bench.py --
    the forward hands the gate kernel's products to the backward in a caller-owned block, and the
    step is captured into a CUDA graph after a warm-up and replayed; the outputs compared are those
    of the replay."""
    w = W.CONFIGS[name]
    x = W.make_inputs(w)
    p = gsa.Params(w.B, w.T, w.H, w.d_k, w.d_v, w.m, io=w.io, tc_operands=tc_operands)
    q, k, v = (to_dev(x[n], w.io) for n in ("q", "k", "v"))
    gate = to_dev(x["gate"])
    K0, V0 = to_dev(x.get("K0")), to_dev(x.get("V0"))
    io = p.io_dtype
    ok = torch.empty(w.B, w.T, w.H, w.m, device="cuda")
    KT = torch.empty(w.B, w.H, w.m, w.d_k, device="cuda")
    VT = torch.empty(w.B, w.H, w.m, w.d_v, device="cuda")
    o = torch.empty(w.B, w.T, w.H, w.d_v, dtype=io, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = dict(o=o, ok=ok, KT=KT, VT=VT)
    dO = to_dev(x["dO"], w.io) if with_bwd else None
    if with_bwd:
        got.update(dq=torch.empty_like(q), dk=torch.empty_like(k), dv=torch.empty_like(v), dgate=torch.empty_like(gate))
    ws_f = torch.empty(gsa.gsa_workspace_bytes(p, 0), dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(gsa.gsa_workspace_bytes(p, 1), dtype=torch.uint8, device="cuda") if with_bwd else None
    blk = gsa.gate_block(p, q.device) if launch == "bench" else None

    def step():
        gsa.gsa_fwd(p, q, k, v, gate, K0, V0, o=o, ok_save=ok, KT=KT, VT=VT, ws=ws_f, dev_status=status,
                    gate_save=blk)
        if with_bwd:
            gsa.gsa_bwd(p, q, k, v, gate, dO, K0, V0, ok_saved=ok, dq=got["dq"], dk=got["dk"], dv=got["dv"],
                        dgate=got["dgate"], ws=ws_b, dev_status=status, gate_saved=blk)

    step()
    torch.cuda.synchronize()
    if launch == "bench":
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        for t in got.values():
            t.zero_()
        graph.replay()
        graph.replay()
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
        kind, limit = TC_CONFIG_BOUNDS[n]
        plain = rel_err(gs, ref[n])
        after = rel_err(gs, ref[n], True)
        errs[n] = dict(bound=after if kind == "bf16out" else plain, plain=plain, limit=limit,
                       after_output_half_ulp=after, plain_ceiling=TC_PLAIN_CEILING.get((name, n)),
                       max_over_rms=float(np.abs(ref[n]).max() / np.sqrt(np.mean(ref[n] ** 2))))
        if n in BF16_IO:
            ulps, equal = bf16_storage_check(gs, ref[n])
            errs[n].update(ulps_from_rounded_oracle=ulps, bit_equal_to_rounded_oracle=equal)
    tag = name + ("" if tc_operands == "paired" else "/" + tc_operands) + ("" if launch == "plain" else "/" + launch)
    record(tag, dict(pairs=pairs, errors=errs))
    print(tag, {n: (round(e["plain"], 5), round(e["bound"], 5), round(e.get("bit_equal_to_rounded_oracle", -1), 4))
                for n, e in errs.items()})
    bad = {}
    for n, e in errs.items():
        if e["bound"] > e["limit"]:
            bad[n] = e
        # the plain figure of a tensor whose storage format alone exceeds the stated bound is held
        # under a recorded ceiling, so that a regression of the arithmetic behind the allowance fails
        if e["plain_ceiling"] is not None and e["plain"] > e["plain_ceiling"]:
            bad[n] = e
        # a bfloat16-stored tensor is the oracle's value rounded to bfloat16, or its neighbour
        if n in BF16_IO and tc_operands == "paired" and (
                e["ulps_from_rounded_oracle"] > 1.0 or e["bit_equal_to_rounded_oracle"] < 0.95):
            bad[n] = e
    assert not bad, bad


@pytest.mark.parametrize("launch", ["plain", "bench"])
def test_config_train_1p3b_fwd_bwd(launch):
    run_training_config("train_1p3b", with_bwd=True, launch=launch)


@pytest.mark.parametrize("launch", ["plain", "bench"])
def test_config_t2r_7b_fwd_bwd(launch):
    run_training_config("t2r_7b", with_bwd=True, launch=launch)


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
