"""The tcgen05 building blocks (TMA tile loads, swizzled operand panels, matrix
descriptors, MMA issue, accumulator loads) on one 128-row product per operand layout."""
import numpy as np
import pytest
import torch

import paper_2409_07146_b200 as gsa

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", [0, 1, 2, 3, 4, 5])
def test_tc_selftest_products(mode):
    g = torch.Generator().manual_seed(mode)
    X = torch.randn(128, 128, generator=g).to(torch.bfloat16)
    Y = torch.randn(128, 128, generator=g).to(torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    D = gsa.gsa_tc_selftest(mode, X.cuda(), Y.cuda(), status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "a bounded wait expired"
    x, y = X.double().numpy(), Y.double().numpy()
    ref = {0: x @ y.T, 1: x @ y, 2: x.T @ y[:64].T, 3: x @ y[:, :64], 4: x @ y.T, 5: x @ y}[mode]
    err = np.abs(D.cpu().double().numpy() - ref).max()
    assert err < 1e-3, err
