"""The fused chunk kernel (pass 1 -> slot softmax -> pass 2 in one kernel, and dp -> dsoftmax ->
dq in the backward; Algorithm 1's driver lines with the slot rows kept on chip) against the
sequential fp64 oracle, for every cluster size it runs with (d / 128 = 1, 2, 4 CTAs per
(batch, head)), ragged lengths, carried memories, the element-wise replacements of the
softmax, and against the separate-kernel path on the same inputs."""
import numpy as np
import pytest
import torch

import oracle
import paper_2409_07146_b200 as gsa
from util import BF16_IO, TOL, bf16_half_ulp, bf16_storage_check, rand_inputs, rel_err, to_dev, to_np

pytestmark = pytest.mark.gpu


def run(d, B, T, H, dk, dv, m, fuse, scale=1.0, act="softmax", saved=True, final_grads=False):
    p = gsa.Params(B, T, H, dk, dv, m, io="bf16", impl="tc", scale=scale, slot_act=act, fuse=fuse)
    q, k, v, dO = (to_dev(d[n], "bf16") for n in ("q", "k", "v", "dO"))
    gate = to_dev(d["gate"])
    K0, V0 = to_dev(d.get("K0")), to_dev(d.get("V0"))
    dKT, dVT = (to_dev(d.get(n)) if final_grads else None for n in ("dKT", "dVT"))
    ok = torch.empty(B, T, H, m, device="cuda")
    KT = torch.empty(B, H, m, dk, device="cuda"); VT = torch.empty(B, H, m, dv, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = gsa.gsa_fwd(p, q, k, v, gate, K0, V0, ok_save=ok, KT=KT, VT=VT, dev_status=status)
    dK0 = torch.empty(B, H, m, dk, device="cuda"); dV0 = torch.empty(B, H, m, dv, device="cuda")
    dq, dk_, dv_, dg = gsa.gsa_bwd(p, q, k, v, gate, dO, K0, V0, ok_saved=ok if saved else None, dKT=dKT, dVT=dVT,
                                   dK0=dK0, dV0=dV0, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "a bounded device-side wait expired"
    return dict(o=to_np(o), ok=to_np(ok), KT=to_np(KT), VT=to_np(VT), dq=to_np(dq), dk=to_np(dk_), dv=to_np(dv_),
                dgate=to_np(dg), dK0=to_np(dK0), dV0=to_np(dV0))


def reference(d, scale=1.0, act="softmax", final_grads=False):
    ref = oracle.fwd(d["q"], d["k"], d["v"], d["gate"], scale=scale, K0=d.get("K0"), V0=d.get("V0"), act=act)
    ref.update(oracle.bwd(d["q"], d["k"], d["v"], d["gate"], d["dO"], scale=scale, K0=d.get("K0"), V0=d.get("V0"),
                          dKT=d.get("dKT") if final_grads else None, dVT=d.get("dVT") if final_grads else None, act=act))
    return ref


def check(got, ref, names=None):
    errs = {n: rel_err(got[n], ref[n], n in BF16_IO) for n in (names or got) if n in ref}
    assert all(np.isfinite(got[n]).all() for n in errs), "non-finite output"
    assert all(e <= TOL["bf16"] for e in errs.values()), errs
    st = {n: bf16_storage_check(got[n], ref[n]) for n in BF16_IO if n in errs}
    assert all(u <= 2.0 and eq >= 0.95 for u, eq in st.values()), st
    return errs


@pytest.mark.parametrize("d", [128, 256, 512])
@pytest.mark.parametrize("T", [1, 100, 128, 129, 300, 640])
def test_fused_fwd_bwd_against_oracle(d, T):
    B, H, m = 2, 2, 64
    x = rand_inputs(1000 + T + d, B, T, H, d, d, m, "bf16", init=True, final_grads=True)
    got = run(x, B, T, H, d, d, m, fuse=True, scale=0.9, final_grads=True)
    errs = check(got, reference(x, scale=0.9, final_grads=True))
    print("fused", d, T, {n: float("%.2g" % e) for n, e in errs.items()})


@pytest.mark.parametrize("d", [128, 512])
def test_fused_agrees_with_separate_kernels(d):
    # same operand roundings in both paths; only the order of a few fp32 additions differs
    B, T, H, m = 2, 520, 3, 64
    x = rand_inputs(77 + d, B, T, H, d, d, m, "bf16", init=True)
    a = run(x, B, T, H, d, d, m, fuse=True)
    b = run(x, B, T, H, d, d, m, fuse=False)
    for n in a:
        if n in BF16_IO:      # the two roundings to bfloat16 may fall on neighbouring values: one ulp apart at most
            rms = np.sqrt(np.mean(b[n] ** 2))      # (small elements: the ulp at 2e-2 of the rms, as in bf16_storage_check)
            assert (np.abs(a[n] - b[n]) <= 2.0 * bf16_half_ulp(np.maximum(np.abs(b[n]), 2e-2 * rms))).all(), n
            assert np.mean(a[n] == b[n]) >= 0.99, n
        else:                 # fp32: the order of a few additions
            assert rel_err(a[n], b[n]) <= 2e-4, n


@pytest.mark.parametrize("saved", [False, True])
def test_fused_without_initial_memories_and_with_recomputed_logits(saved):
    B, T, H, d, m = 1, 384, 2, 256, 64
    x = rand_inputs(55, B, T, H, d, d, m, "bf16")
    got = run(x, B, T, H, d, d, m, fuse=True, saved=saved)
    check(got, reference(x))


@pytest.mark.parametrize("act", ["none", "relu", "swish", "relu2"])
def test_fused_slot_activation_variants(act):
    B, T, H, d, m = 2, 300, 2, 256, 64
    x = rand_inputs(91, B, T, H, d, d, m, "bf16", init=True)
    got = run(x, B, T, H, d, d, m, fuse=True, scale=0.5, act=act)
    check(got, reference(x, scale=0.5, act=act))


def test_fused_is_deterministic():
    B, T, H, d, m = 2, 300, 2, 512, 64
    x = rand_inputs(5, B, T, H, d, d, m, "bf16", init=True)
    a = run(x, B, T, H, d, d, m, fuse=True)
    b = run(x, B, T, H, d, d, m, fuse=True)
    for n in a:
        np.testing.assert_array_equal(a[n], b[n])


def test_fused_forward_without_saved_logits_writes_no_logits():
    # ok_save == NULL: the logits exist on chip only; o must be what the saving call gives
    B, T, H, d, m = 1, 260, 2, 512, 64
    x = rand_inputs(6, B, T, H, d, d, m, "bf16")
    p = gsa.Params(B, T, H, d, d, m, io="bf16", impl="tc")
    q, k, v = (to_dev(x[n], "bf16") for n in ("q", "k", "v"))
    gate = to_dev(x["gate"])
    ok = torch.empty(B, T, H, m, device="cuda")
    o1 = gsa.gsa_fwd(p, q, k, v, gate, ok_save=ok)
    o2 = gsa.gsa_fwd(p, q, k, v, gate)
    torch.cuda.synchronize()
    assert torch.equal(o1, o2)
