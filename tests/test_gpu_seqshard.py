"""Sequence sharding on the GPU: the sharding driver over the CUDA library (gsa_shard_states,
gsa_shard_combine, gsa_fwd, gsa_bwd through the C ABI), with three ranks played one GPU by three
host threads that exchange their shard memories in process (no kernel waits on another: the
exchange is a host-side hand-over), against the oracle on the whole sequence."""
import numpy as np
import pytest
import torch

import oracle
import paper_2409_07146_b200 as gsa
from paper_2409_07146_b200 import seqshard
from seqshard_util import run_ranks_as_threads
from util import BF16_IO, TOL, rand_inputs, rel_err, to_dev, to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("io,impl,Ts,d", [("f32", "auto", 100, 64), ("bf16", "tc", 256, 128), ("bf16", "tc", 200, 256)])
def test_three_shards_on_one_gpu_match_the_whole_sequence(io, impl, Ts, d):
    world, B, H, m = 3, 2, 2, 64
    T = world * Ts
    x = rand_inputs(70 + Ts, B, T, H, d, d, m, io, init=True, final_grads=True)
    ref = oracle.fwd(x["q"], x["k"], x["v"], x["gate"], K0=x["K0"], V0=x["V0"])
    ref.update(oracle.bwd(x["q"], x["k"], x["v"], x["gate"], x["dO"], K0=x["K0"], V0=x["V0"], dKT=x["dKT"], dVT=x["dVT"]))
    K0, V0, dKT, dVT = (to_dev(x[n]) for n in ("K0", "V0", "dKT", "dVT"))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def rank_fn(rank, gather):
        torch.cuda.set_device(0)
        lo, hi = rank * Ts, (rank + 1) * Ts
        xs = {n: to_dev(x[n][:, lo:hi], io) for n in ("q", "k", "v")}
        xs["gate"] = to_dev(x["gate"][:, lo:hi])
        dO = to_dev(x["dO"][:, lo:hi], io)
        p = gsa.Params(B, Ts, H, d, d, m, io=io, impl=impl)
        eng = seqshard.CudaEngine(p, dev_status=status)
        o, saved = seqshard.sharded_forward(eng, gather, rank, xs, d, d, K0, V0)
        g = seqshard.sharded_backward(eng, gather, rank, xs, dO, saved, d, d, dKT, dVT)
        torch.cuda.synchronize()
        return dict(o=to_np(o), KT=to_np(saved["KT"]), VT=to_np(saved["VT"]), **{n: to_np(v) for n, v in g.items()})

    parts = run_ranks_as_threads(world, rank_fn)
    assert int(status.item()) == 0
    errs = {}
    for n in ("o", "dq", "dk", "dv", "dgate"):
        got = np.concatenate([p[n] for p in parts], axis=1)
        errs[n] = rel_err(got, ref[n], io == "bf16" and n in BF16_IO)
    for n in ("KT", "VT", "dK0", "dV0"):
        errs[n] = max(rel_err(p[n], ref[n]) for p in parts)
    print("seqshard gpu", io, Ts, d, {n: float("%.2g" % e) for n, e in errs.items()})
    assert all(e <= TOL[io] for e in errs.values()), errs
