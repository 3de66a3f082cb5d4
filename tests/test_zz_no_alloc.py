"""gsa_fwd_noalloc, the forward for callers that cannot allocate device memory (a server
with a fixed memory plan, a real-time loop, a plug-in that only gets input and output
buffers): its scratch is a fixed array inside the library.  Called through the C ABI, it
must give what gsa_fwd gives, on two calls in a row that reuse the array.  Collected last
on purpose (file name), so that a failure here cannot hide the other tests."""
import numpy as np
import pytest
import torch

import oracle
import paper_2409_07146_b200 as gsa
from util import TOL, rand_inputs, rel_err, to_dev

pytestmark = pytest.mark.gpu


def _run_both(seed, B, T, H, dk, dv, m, io):
    d = rand_inputs(seed, B, T, H, dk, dv, m, io, init=True)
    p = gsa.Params(B, T, H, dk, dv, m, io=io)
    q, k, v = (to_dev(d[n], io) for n in ("q", "k", "v"))
    gate, K0, V0 = to_dev(d["gate"]), to_dev(d["K0"]), to_dev(d["V0"])

    def outputs():
        return dict(o=torch.empty(B, T, H, dv, dtype=p.io_dtype, device="cuda"),
                    ok_save=torch.empty(B, T, H, m, device="cuda"),
                    KT=torch.empty(B, H, m, dk, device="cuda"), VT=torch.empty(B, H, m, dv, device="cuda"))

    ref, got = outputs(), outputs()
    gsa.gsa_fwd(p, q, k, v, gate, K0, V0, **ref)
    gsa.gsa_fwd_noalloc(p, q, k, v, gate, K0=K0, V0=V0, **got)
    torch.cuda.synchronize()
    for n in ref:
        a, b = ref[n].float().cpu().numpy(), got[n].float().cpu().numpy()
        assert np.isfinite(b).all(), n
        # same kernels, same order, same inputs: the two entry points must agree to the bit
        np.testing.assert_array_equal(a, b, err_msg=n)
    # ... and these shapes and seeds against the oracle itself
    want = oracle.fwd(d["q"], d["k"], d["v"], d["gate"], K0=d["K0"], V0=d["V0"])
    for n, name in (("o", "o"), ("ok_save", "ok"), ("KT", "KT"), ("VT", "VT")):
        e = rel_err(got[n].float().cpu().numpy(), want[name], io == "bf16" and n == "o")
        assert e <= TOL[io], (n, e)


def test_noalloc_forward_matches_gsa_fwd_twice_in_a_row():
    # two calls back to back share the built-in scratch: the second (another shape, another
    # kernel family) must not see anything of the first
    _run_both(901, 2, 300, 2, 128, 128, 64, "bf16")     # tensor-core kernels
    _run_both(902, 1, 200, 3, 64, 128, 32, "f32")       # fp32 CUDA-core kernels
    _run_both(903, 2, 300, 2, 128, 128, 64, "bf16")


def test_noalloc_steady_state_call_leaves_device_memory_alone():
    # after the first call on this device (symbol lookup, the library's side stream and events) a
    # call must not change the amount of free device memory
    p = gsa.Params(2, 300, 2, 128, 128, 64, io="bf16")
    d = rand_inputs(904, 2, 300, 2, 128, 128, 64, "bf16")
    q, k, v = (to_dev(d[n], "bf16") for n in ("q", "k", "v"))
    gate = to_dev(d["gate"])
    o = torch.empty(2, 300, 2, 128, dtype=torch.bfloat16, device="cuda")
    gsa.gsa_fwd_noalloc(p, q, k, v, gate, o=o)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0 = torch.cuda.memory_allocated()
    for _ in range(3):
        gsa.gsa_fwd_noalloc(p, q, k, v, gate, o=o)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0


def test_noalloc_rejects_shapes_beyond_its_scratch():
    big = gsa.Params(8, 2048, 4, 512, 512, 64, io="bf16")
    assert gsa.gsa_workspace_bytes(big, 0) > gsa.GSA_NOALLOC_MAX_WORKSPACE_BYTES
    x = torch.zeros(8, dtype=torch.float32, device="cuda")
    import ctypes
    cp = big.c()
    lib = gsa.load_library()
    ptr = ctypes.c_void_p(x.data_ptr())
    rc = lib.gsa_fwd_noalloc(ctypes.byref(cp), ptr, ptr, ptr, ptr, None, None, ptr, None, None, None, None, None)
    assert rc == 3 and lib.gsa_status_string(rc).decode().startswith("workspace")
