"""Sequence sharding of the GSA layer across ranks (one sequence cut into R shards along T, one
per GPU): the order of the local steps and of the one exchange they need.

The memories of Eq. 6 are linear in (k, v): the memory after a stretch of tokens is
D * (memory before) + (memory of the stretch run from empty memories), with D the product of the
stretch's gates.  So every rank needs from the others only their shards' end memories and
log-decays -- m (d_k + d_v + 1) floats per (batch, head) -- gathered once into local memory; the
token-sized tensors never leave their GPU.  The backward needs the mirror image for the memory
gradients, which are linear too.

This module holds no arithmetic: `engine` does the local work (the CUDA library through its C ABI,
`CudaEngine` below; the tests run the same driver over the fp64 oracle on CPU ranks), `gather`
does the exchange (torch.distributed.all_gather over NCCL or gloo; a list concatenation when one
process emulates the ranks one after the other).
"""
from __future__ import annotations


def dist_gather(t):
    """all_gather of one tensor over the default process group -> [R, ...] in rank order."""
    import torch
    import torch.distributed as dist
    out = [torch.empty_like(t) for _ in range(dist.get_world_size())]
    dist.all_gather(out, t.contiguous())
    return torch.stack(out)


class CudaEngine:
    """The local steps on this rank's GPU, through the C-ABI binding."""

    def __init__(self, params, dev_status=None):
        from . import binding
        self.b = binding
        self.p = params
        self.dev_status = dev_status

    def states(self, x):
        return self.b.gsa_shard_states(self.p, x["k"], x["v"], x["gate"], dev_status=self.dev_status)

    def combine(self, d, rank, logdecay_all, local_all, S0=None, reverse=False, want_final=False):
        return self.b.gsa_shard_combine(self.p, d, rank, logdecay_all, local_all, S0, reverse, want_final)

    def fwd(self, x, K0, V0):
        import torch
        ok = torch.empty(self.p.B, self.p.T, self.p.H, self.p.m, dtype=torch.float32, device=x["q"].device)
        o = self.b.gsa_fwd(self.p, x["q"], x["k"], x["v"], x["gate"], K0, V0, ok_save=ok, dev_status=self.dev_status)
        return o, ok

    def bwd(self, x, dO, K0, V0, ok, dKT, dVT):
        import torch
        dK0 = torch.empty(self.p.B, self.p.H, self.p.m, self.p.d_k, dtype=torch.float32, device=dO.device)
        dV0 = torch.empty(self.p.B, self.p.H, self.p.m, self.p.d_v, dtype=torch.float32, device=dO.device)
        dq, dk, dv, dg = self.b.gsa_bwd(self.p, x["q"], x["k"], x["v"], x["gate"], dO, K0, V0, ok_saved=ok, dKT=dKT,
                                        dVT=dVT, dK0=dK0, dV0=dV0, dev_status=self.dev_status)
        return dict(dq=dq, dk=dk, dv=dv, dgate=dg, dK0=dK0, dV0=dV0)


def sharded_forward(engine, gather, rank, x, d_k, d_v, K0=None, V0=None):
    """Forward of this rank's shard x = {q, k, v, gate}.  K0 / V0: the memories before the FIRST shard
    (every rank passes the same).  Returns (o, saved) where saved carries what the backward reuses; on
    every rank saved["KT"] / saved["VT"] are the memories after the LAST shard."""
    Kloc, Vloc, logd = engine.states(x)
    logd_all, K_all, V_all = gather(logd), gather(Kloc), gather(Vloc)
    Kin, KT = engine.combine(d_k, rank, logd_all, K_all, K0, want_final=True)
    Vin, VT = engine.combine(d_v, rank, logd_all, V_all, V0, want_final=True)
    o, ok = engine.fwd(x, Kin, Vin)
    return o, dict(Kin=Kin, Vin=Vin, ok=ok, logdecay_all=logd_all, KT=KT, VT=VT)


def sharded_backward(engine, gather, rank, x, dO, saved, d_k, d_v, dKT=None, dVT=None):
    """Backward of this rank's shard.  dKT / dVT: gradients w.r.t. the memories after the LAST shard
    (every rank passes the same).  Two local backward runs: the first with zero final-memory gradients
    gives the shard's own contribution to the gradient of the memories that enter it (that gradient is
    linear in what arrives from the right), the exchange turns the contributions into the gradient
    arriving at every shard from the right, the second run uses it.  Returns the gradients of the
    shard's tokens; dK0 / dV0 are those of the memories before the FIRST shard on every rank."""
    first = engine.bwd(x, dO, saved["Kin"], saved["Vin"], saved["ok"], None, None)
    dK_all, dV_all = gather(first["dK0"]), gather(first["dV0"])
    logd_all = saved["logdecay_all"]
    dKend, dK0 = engine.combine(d_k, rank, logd_all, dK_all, dKT, reverse=True, want_final=True)
    dVend, dV0 = engine.combine(d_v, rank, logd_all, dV_all, dVT, reverse=True, want_final=True)
    R = logd_all.shape[0]
    if rank == R - 1 and dKT is None and dVT is None:
        out = first                       # nothing arrives at the last shard: its first run is final
    else:
        out = engine.bwd(x, dO, saved["Kin"], saved["Vin"], saved["ok"], dKend, dVend)
    out = dict(out)
    out["dK0"], out["dV0"] = dK0, dV0
    return out
