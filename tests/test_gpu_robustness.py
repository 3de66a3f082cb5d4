"""Stand-ins for a memory checker and for fault injection on the device, none of which faults,
traps or hangs the GPU: a bounded wait that is made to expire (an mbarrier nothing signals, a
limit of a few milliseconds) must report GSA_ERR_TIMEOUT and leave the context usable; outputs
and workspace framed by guard bands must come back with the bands intact; the library's
internal streams can be released and come back on demand."""
import numpy as np
import pytest
import torch

import gsa_workloads as W
import oracle
import paper_2409_07146_b200 as gsa
from util import TOL, rand_inputs, rel_err, to_dev, to_np

pytestmark = pytest.mark.gpu

GUARD = 4096          # bytes of guard band on either side of a buffer
PATTERN = 0xA5


class Guarded:
    """A device buffer of `nbytes` bytes with a guard band before and after it, 256-byte aligned."""

    def __init__(self, nbytes):
        self.nbytes = nbytes
        self.pad = (nbytes + 255) // 256 * 256
        self.raw = torch.full((GUARD + self.pad + GUARD,), PATTERN, dtype=torch.uint8, device="cuda")

    def view(self, dtype, shape):
        return self.raw[GUARD:GUARD + self.nbytes].view(dtype).view(*shape)

    def bytes(self):
        return self.raw[GUARD:GUARD + self.pad]

    def intact(self):
        head, tail = self.raw[:GUARD], self.raw[GUARD + self.pad:]
        return bool((head == PATTERN).all()) and bool((tail == PATTERN).all())


def guarded_like(shape, dtype):
    n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
    g = Guarded(n)
    return g, g.view(dtype, shape)


def test_bounded_wait_expires_cleanly_and_the_context_stays_usable():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    waited = torch.zeros(1, dtype=torch.int32, device="cuda")
    gsa.gsa_wait_selftest(3000, status, waited)          # 3 ms on a barrier nobody arrives at
    torch.cuda.synchronize()
    assert int(status.item()) == 5                        # GSA_ERR_TIMEOUT
    assert 2500 <= int(waited.item()) <= 100000, int(waited.item())
    assert gsa.load_library().gsa_status_string(5).decode().startswith("bounded")
    # the same context runs the tensor-core forward right after, and it matches the oracle
    B, T, H, d, m = 1, 300, 2, 128, 64
    x = rand_inputs(3, B, T, H, d, d, m, "bf16")
    p = gsa.Params(B, T, H, d, d, m, io="bf16", impl="tc")
    st2 = torch.zeros(1, dtype=torch.int32, device="cuda")
    o = gsa.gsa_fwd(p, to_dev(x["q"], "bf16"), to_dev(x["k"], "bf16"), to_dev(x["v"], "bf16"), to_dev(x["gate"]),
                    dev_status=st2)
    torch.cuda.synchronize()
    assert int(st2.item()) == 0
    ref = oracle.fwd(x["q"], x["k"], x["v"], x["gate"])
    assert rel_err(to_np(o), ref["o"], True) <= TOL["bf16"]


@pytest.mark.parametrize("io,impl,T", [("bf16", "tc", 300), ("f32", "auto", 150), ("bf16", "tc", 4096)])
def test_forward_and_backward_stay_inside_their_buffers(io, impl, T):
    B, H, d, m = (1, 1, 128, 64) if T == 4096 else (2, 2, 128, 64)     # T = 4096, one pair: segment-parallel scheduling
    x = rand_inputs(11 + T, B, T, H, d, d, m, io, init=True, final_grads=True)
    p = gsa.Params(B, T, H, d, d, m, io=io, impl=impl)
    q, k, v, dO = (to_dev(x[n], io) for n in ("q", "k", "v", "dO"))
    gate, K0, V0, dKT, dVT = (to_dev(x[n]) for n in ("gate", "K0", "V0", "dKT", "dVT"))
    iot = p.io_dtype
    bufs = {}

    def out(name, shape, dtype):
        g, t = guarded_like(shape, dtype)
        bufs[name] = g
        return t

    o = out("o", (B, T, H, d), iot); ok = out("ok", (B, T, H, m), torch.float32)
    KT = out("KT", (B, H, m, d), torch.float32); VT = out("VT", (B, H, m, d), torch.float32)
    dq = out("dq", (B, T, H, d), iot); dk = out("dk", (B, T, H, d), iot); dv = out("dv", (B, T, H, d), iot)
    dg = out("dgate", (B, T, H, m), torch.float32)
    dK0 = out("dK0", (B, H, m, d), torch.float32); dV0 = out("dV0", (B, H, m, d), torch.float32)
    ws_f = Guarded(gsa.gsa_workspace_bytes(p, 0)); ws_b = Guarded(gsa.gsa_workspace_bytes(p, 1))
    bufs["ws_fwd"], bufs["ws_bwd"] = ws_f, ws_b
    gsa.gsa_fwd(p, q, k, v, gate, K0, V0, o=o, ok_save=ok, KT=KT, VT=VT, ws=ws_f.bytes())
    gsa.gsa_bwd(p, q, k, v, gate, dO, K0, V0, ok_saved=ok, dKT=dKT, dVT=dVT, dq=dq, dk=dk, dv=dv, dgate=dg, dK0=dK0,
                dV0=dV0, ws=ws_b.bytes())
    torch.cuda.synchronize()
    broken = [n for n, g in bufs.items() if not g.intact()]
    assert not broken, broken
    ref = oracle.bwd(x["q"], x["k"], x["v"], x["gate"], x["dO"], K0=x["K0"], V0=x["V0"], dKT=x["dKT"], dVT=x["dVT"])
    assert rel_err(to_np(dg), ref["dgate"]) <= TOL[io]      # ... and the call still computed the right thing


def test_decode_stays_inside_its_buffers():
    S, H, d, m = 5, 3, 128, 64
    w = W.CONFIGS["decode"].scaled(B=S, H=H, d_k=d, d_v=d, m=m)
    st = W.make_decode_states(w)
    gK, Ks = guarded_like((S, H, m, d), torch.float32)
    gV, Vs = guarded_like((S, H, m, d), torch.float32)
    go, o = guarded_like((S, H, d), torch.bfloat16)
    Ks.copy_(to_dev(st["K"])); Vs.copy_(to_dev(st["V"]))
    Kr, Vr = st["K"].astype(np.float64), st["V"].astype(np.float64)
    p = gsa.Params(S, 1, H, d, d, m, io="bf16")
    for step in range(2):
        x = W.make_decode_step_inputs(w, step)
        gsa.gsa_decode_step(p, to_dev(x["q"], "bf16"), to_dev(x["k"], "bf16"), to_dev(x["v"], "bf16"), to_dev(x["gate"]),
                            Ks, Vs, o=o)
        ro = oracle.decode_step(x["q"], x["k"], x["v"], x["gate"], Kr, Vr)
    torch.cuda.synchronize()
    assert gK.intact() and gV.intact() and go.intact()
    assert rel_err(to_np(o), ro, True) <= TOL["bf16"] and rel_err(to_np(Ks), Kr) <= 1e-5


def test_internal_streams_can_be_released_and_come_back():
    B, T, H, d, m = 1, 200, 2, 128, 64
    x = rand_inputs(8, B, T, H, d, d, m, "bf16")
    p = gsa.Params(B, T, H, d, d, m, io="bf16", impl="tc")
    args = [to_dev(x[n], "bf16") for n in ("q", "k", "v")] + [to_dev(x["gate"])]
    a = gsa.gsa_fwd(p, *args)
    torch.cuda.synchronize()
    gsa.gsa_release_streams()
    gsa.gsa_release_streams()          # nothing left to release: still fine
    b = gsa.gsa_fwd(p, *args)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
