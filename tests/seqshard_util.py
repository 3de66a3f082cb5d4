"""Test-side pieces for the sequence-sharding driver: an engine that does the local steps with the
fp64 oracle (so the driver's order of steps and exchanges can be checked on CPU ranks), and an
in-process stand-in for the all-gather (threads as ranks)."""
import threading

import numpy as np
import torch

import oracle


class OracleEngine:
    """The driver's local steps in fp64 on the CPU: oracle calls plus the textbook combination
    S_in(r) = D_{r-1} S_in(r-1) + S_loc(r-1) written out in numpy."""

    def __init__(self, scale=1.0):
        self.scale = scale

    @staticmethod
    def _np(t):
        return None if t is None else t.numpy()

    def states(self, x):
        r = oracle.fwd(self._np(x["q"]), self._np(x["k"]), self._np(x["v"]), self._np(x["gate"]), scale=self.scale)
        logd = np.log(np.maximum(self._np(x["gate"]).astype(np.float64), 1e-300)).sum(axis=1)      # [B,H,m]
        return torch.from_numpy(r["KT"]), torch.from_numpy(r["VT"]), torch.from_numpy(logd)

    def combine(self, d, rank, logdecay_all, local_all, S0=None, reverse=False, want_final=False):
        R = logdecay_all.shape[0]
        cur = np.zeros(local_all.shape[1:]) if S0 is None else S0.numpy().astype(np.float64)
        start = None
        for i in range(R):
            r = R - 1 - i if reverse else i
            if r == rank:
                start = cur.copy()
            cur = cur * np.exp(logdecay_all[r].numpy())[..., None] + local_all[r].numpy()
        start = torch.from_numpy(start)
        return (start, torch.from_numpy(cur)) if want_final else start

    def fwd(self, x, K0, V0):
        r = oracle.fwd(self._np(x["q"]), self._np(x["k"]), self._np(x["v"]), self._np(x["gate"]), scale=self.scale,
                       K0=self._np(K0), V0=self._np(V0))
        return torch.from_numpy(r["o"]), torch.from_numpy(r["ok"])

    def bwd(self, x, dO, K0, V0, ok, dKT, dVT):
        r = oracle.bwd(self._np(x["q"]), self._np(x["k"]), self._np(x["v"]), self._np(x["gate"]), self._np(dO),
                       scale=self.scale, K0=self._np(K0), V0=self._np(V0), dKT=self._np(dKT), dVT=self._np(dVT))
        return {n: torch.from_numpy(np.ascontiguousarray(v)) for n, v in r.items()}


class ThreadGather:
    """all_gather among R threads of one process (each thread plays a rank)."""

    def __init__(self, world):
        self.world = world
        self.slots = [None] * world
        self.barrier = threading.Barrier(world)

    def bind(self, rank):
        def gather(t):
            self.slots[rank] = t
            self.barrier.wait()
            out = torch.stack([s.clone() for s in self.slots])
            self.barrier.wait()
            return out
        return gather


def run_ranks_as_threads(world, fn):
    """fn(rank, gather) on `world` threads; returns the per-rank results, re-raising the first error."""
    tg = ThreadGather(world)
    results, errors = [None] * world, []

    def work(r):
        try:
            results[r] = fn(r, tg.bind(r))
        except BaseException as exc:      # noqa: BLE001
            errors.append(exc)
            tg.barrier.abort()

    threads = [threading.Thread(target=work, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    if errors:
        raise errors[0]
    return results
