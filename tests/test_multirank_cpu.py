"""The N > 1 path on CPU: two gloo ranks.  The layer shards over batch with no data-path
collective; what the ranks share is a barrier and the max-over-ranks time.  Here each rank
runs the fp64 oracle on its own batch shard and the gathered shards must equal one
single-process run; the timing reduction and the rank seeding of bench.py are exercised too."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
import gsa_workloads as W
import oracle


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.CONFIGS["tiny_f32"].scaled(B=4, T=40)
        x = W.make_inputs(w)
        lo, hi = rank * w.B // world, (rank + 1) * w.B // world      # this rank's batch shard
        part = oracle.fwd(x["q"][lo:hi], x["k"][lo:hi], x["v"][lo:hi], x["gate"][lo:hi], threads=1)
        gathered = [None] * world
        dist.all_gather_object(gathered, part["o"])
        slow = bench.max_over_ranks(10.0 + rank, world)               # the slowest rank decides
        seeds = [None] * world
        dist.all_gather_object(seeds, bench.rank_workload(rank).seed)
        dist.barrier()
        if rank == 0:
            np.save(os.path.join(out_dir, "o.npy"), np.concatenate(gathered, 0))
            np.save(os.path.join(out_dir, "meta.npy"), np.array([slow] + seeds, dtype=np.float64))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_the_batch(tmp_path):
    oracle.build()
    world, port = 2, _free_port()
    mp.start_processes(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True,
                       start_method="spawn")
    w = W.CONFIGS["tiny_f32"].scaled(B=4, T=40)
    x = W.make_inputs(w)
    full = oracle.fwd(x["q"], x["k"], x["v"], x["gate"], threads=1)
    np.testing.assert_array_equal(np.load(tmp_path / "o.npy"), full["o"])
    meta = np.load(tmp_path / "meta.npy")
    assert meta[0] == 11.0                       # max over ranks of (10, 11)
    assert meta[1] != meta[2]                    # every rank draws its own batch
    assert bench.aggregate_tokens_per_s(2, 16384, 1.0) == 2 * 16384 / 1e-3


def test_bench_starts_its_own_ranks_when_run_as_a_plain_process(tmp_path):
    """`python bench.py --gpus 2` without a launcher must start two ranks itself and print one line with
    n_gpus = 2.  Exercised here on the reference arm (the oracle on CPU: rank 0 works, rank 1 exits 0)."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    cmd = bench.launcher_command(2, ["--gpus", "2"])
    assert "--nproc-per-node=2" in cmd and "127.0.0.1" in cmd and cmd[-2:] == ["--gpus", "2"]
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--impl", "reference",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2


def test_bench_byte_model_knows_every_step_label():
    """Every timing label that a training step of the library can emit (the GSA_LAUNCH names of the forward
    and backward cores) has an entry in bench.py's byte model: a new kernel must not break the bench line."""
    import re
    import gsa_workloads as W
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = open(os.path.join(root, "paper_2409_07146_b200", "csrc", "api.cu")).read()
    labels = set(re.findall(r'GSA_LAUNCH\("([a-zA-Z0-9_]+)"', src))
    step = {l for l in labels if l.startswith(("pass1", "pass2", "bwd_", "slot_softmax", "gate_cumsum", "gate_grad", "fused_"))}
    assert {"pass1_value_side", "pass2_key_side", "bwd_dv_dIv_pair_rev", "bwd_dk_dIk_pair_rev", "gate_grad"} <= step
    w = W.CONFIGS["train_1p3b"]
    for lab in sorted(step):
        assert bench.kernel_algorithmic_bytes(lab, w) > 0, lab
        assert isinstance(bench.kernel_function(lab), str)
