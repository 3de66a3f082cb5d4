"""gsa_fwd_noalloc, the forward for callers that cannot allocate device memory (a server
with a fixed memory plan, a real-time loop, a plug-in that only gets input and output
buffers): its scratch is a fixed array inside the library.  Called through the C ABI, it
must give what gsa_fwd gives, on two calls in a row that reuse the array.  Collected last
on purpose (file name), so that a failure here cannot hide the other tests."""
import numpy as np
import pytest
import torch

import paper_2409_07146_b200 as gsa
from util import rand_inputs, to_dev

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


def test_noalloc_forward_matches_gsa_fwd_twice_in_a_row():
    # two calls back to back share the built-in scratch: the second (another shape, another
    # kernel family) must not see anything of the first
    _run_both(901, 2, 300, 2, 128, 128, 64, "bf16")     # tensor-core kernels
    _run_both(902, 1, 200, 3, 64, 128, 32, "f32")       # fp32 CUDA-core kernels
    _run_both(903, 2, 300, 2, 128, 128, 64, "bf16")


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
