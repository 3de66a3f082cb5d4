"""Sequence sharding across ranks on CPU: two gloo ranks each hold half of every sequence, run
the sharding driver (paper_2409_07146_b200/seqshard.py) with the oracle doing the local steps,
exchange the shard memories with torch.distributed.all_gather, and must reproduce the
single-process oracle on the whole sequence -- outputs, every gradient, the gradients of the
initial memories and the final memories (the state-carry identity of Eq. 6 and its mirror image
for the memory gradients).  A three-rank run with threads as ranks covers a middle shard."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import gsa_workloads as W
import oracle
from paper_2409_07146_b200 import seqshard
from seqshard_util import OracleEngine, run_ranks_as_threads


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _inputs(T):
    w = W.CONFIGS["tiny_f32"].scaled(B=2, T=T, H=2, d_k=8, d_v=16, m=4, init_state=True)
    x = W.make_inputs(w)
    r = np.random.default_rng(9)
    x["dKT"] = r.standard_normal(x["K0"].shape).astype(np.float32)
    x["dVT"] = r.standard_normal(x["V0"].shape).astype(np.float32)
    return w, x


def _shard(x, rank, world, T):
    lo, hi = rank * T // world, (rank + 1) * T // world
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a))
    xs = {n: t(x[n][:, lo:hi]) for n in ("q", "k", "v", "gate")}
    return xs, t(x["dO"][:, lo:hi])


def _run_rank(rank, world, gather, T):
    w, x = _inputs(T)
    xs, dO = _shard(x, rank, world, T)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a))
    eng = OracleEngine()
    o, saved = seqshard.sharded_forward(eng, gather, rank, xs, w.d_k, w.d_v, t(x["K0"]), t(x["V0"]))
    g = seqshard.sharded_backward(eng, gather, rank, xs, dO, saved, w.d_k, w.d_v, t(x["dKT"]), t(x["dVT"]))
    return dict(o=o.numpy(), KT=saved["KT"].numpy(), VT=saved["VT"].numpy(), **{n: v.numpy() for n, v in g.items()})


def _check_against_whole_sequence(parts, T):
    w, x = _inputs(T)
    ref = oracle.fwd(x["q"], x["k"], x["v"], x["gate"], K0=x["K0"], V0=x["V0"])
    ref.update(oracle.bwd(x["q"], x["k"], x["v"], x["gate"], x["dO"], K0=x["K0"], V0=x["V0"], dKT=x["dKT"], dVT=x["dVT"]))
    for n in ("o", "dq", "dk", "dv", "dgate"):
        np.testing.assert_allclose(np.concatenate([p[n] for p in parts], axis=1), ref[n], rtol=1e-9, atol=1e-11, err_msg=n)
    for p in parts:          # every rank ends up with the same final memories and initial-memory gradients
        for n in ("KT", "VT", "dK0", "dV0"):
            np.testing.assert_allclose(p[n], ref[n], rtol=1e-9, atol=1e-11, err_msg=n)


def _worker(rank, world, port, out_dir, T):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        res = _run_rank(rank, world, seqshard.dist_gather, T)
        np.savez(os.path.join(out_dir, f"rank{rank}.npz"), **res)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_the_sequence(tmp_path):
    oracle.build()
    world, T = 2, 48
    mp.start_processes(_worker, args=(world, _free_port(), str(tmp_path), T), nprocs=world, join=True, start_method="spawn")
    parts = [dict(np.load(tmp_path / f"rank{r}.npz")) for r in range(world)]
    _check_against_whole_sequence(parts, T)


def test_three_shards_with_a_middle_rank():
    oracle.build()
    world, T = 3, 45
    parts = run_ranks_as_threads(world, lambda r, gather: _run_rank(r, world, gather, T))
    _check_against_whole_sequence(parts, T)
