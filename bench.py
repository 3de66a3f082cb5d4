#!/usr/bin/env python
"""Benchmark of the GSA layer hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one pass of the whole training hot path over one batch of the 1.3B-model layer
shape (B=8, H=4, T=2048, d_k=d_v=512, m=64, bf16): gsa_fwd (gate cumsum, pass 1, slot
softmax, pass 2, logits saved) followed by gsa_bwd (all gradients).  One JSON line is
printed by rank 0.  With N > 1 (torchrun) every rank runs its own batch (weak scaling, no
data-path collective: (batch, head) pairs are independent recurrences).

--impl reference times the fp64 CPU oracle on the host cores on a bounded sample of the
same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gsa_workloads as W  # noqa: E402

METRIC = "GSA layer fwd+bwd tokens/s (bf16, T=2048, m=64)"
UNIT = "tokens/s"
WORKLOAD = "train_1p3b"


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the tensor-core kernels on this
# workload, from one `ncu --set full` capture (profiles/step_kernels_train_1p3b_ncu_full.md).
NCU_TRAFFIC = {
    "pass1_value_side": 187423232, "bwd_dp_value_side": 186575872,
    "bwd_dIv_value_side_rev": 188858112, "bwd_dIk_value_side_rev": 187463680,
    "pass2_key_side": 130322432, "bwd_dq_key_side": 135258368,
    "bwd_dv_key_side_rev": 130483200, "bwd_dk_key_side_rev": 132975616,
    "bwd_dv_dIv_pair_rev": 258483968, "bwd_dk_dIk_pair_rev": 257145344,
    "gate_cumsum": 17926144, "slot_softmax": 92744448, "slot_softmax_bwd": 118787072,
    "gate_grad": 231503872,     # local + scan + carry
}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d.get("bf16_tflops_sustained", 1400.0)),
                    source="measured (MEASURED_PEAKS.json)")
    return dict(hbm_gbs=6650.0, bf16_tflops=1400.0, source="fallback (profiling recipe)")


# ----------------------------------------------------------------------------- byte model
def step_algorithmic_bytes(w: W.Workload) -> int:
    """Bytes one fwd+bwd step must move if every tensor crossed HBM exactly once: forward
    reads q,k,v,gate and writes o and the saved logits; backward reads q,k,v,dO,gate and the
    saved logits and writes dq,dk,dv,dgate."""
    e = 2 if w.io == "bf16" else 4
    R = w.B * w.T * w.H
    fwd = e * (2 * w.d_k + 2 * w.d_v) + 4 * w.m + 4 * w.m
    bwd = e * (2 * w.d_k + 2 * w.d_v) + e * (2 * w.d_k + w.d_v) + 4 * w.m * 3
    return R * (fwd + bwd)


def kernel_algorithmic_bytes(label: str, w: W.Workload) -> int:
    """Inputs read once plus outputs written once, per launch of each kernel."""
    e = 2 if w.io == "bf16" else 4
    R = w.B * w.T * w.H
    m = w.m
    nsk, nsv = w.d_k // 128, w.d_v // 128
    # bytes per token-head row on the tensor-core path: fp32 [.., m] tensors are 4m, a decayed
    # bf16 operand row [high | residual] is 4m too
    table = {
        "gate_cumsum": 16 * m,                                       # gate -> G, I, I exp(-G)
        "pass1_value_side": 2 * w.d_k * e + 4 * m + 4 * m * nsk,     # q, k, I exp(-G) -> slices of o'
        "slot_softmax": 4 * m * nsk + 12 * m,                        # slices, G -> o', p exp(G)
        "pass2_key_side": 2 * w.d_v * e + 8 * m,                     # v, two decayed rows -> o
        "bwd_dp_value_side": 2 * w.d_v * e + 4 * m + 4 * m * nsv,
        "slot_softmax_bwd": 4 * m * nsv + 20 * m,                    # o', slices, G -> u, p exp(G), dz exp(G)
        "bwd_dq_key_side": 2 * w.d_k * e + 8 * m,
        "bwd_dv_key_side_rev": 2 * w.d_v * e + 8 * m,
        "bwd_dIv_value_side_rev": 2 * w.d_v * e + 4 * m + 4 * m * nsv,
        "bwd_dk_key_side_rev": 2 * w.d_k * e + 8 * m,
        "bwd_dIk_value_side_rev": 2 * w.d_k * e + 4 * m + 4 * m * nsk,
        # a pair of reversed scans as one kernel: both d-sized tiles and both decayed rows once
        "bwd_dv_dIv_pair_rev": 3 * w.d_v * e + 8 * m + 4 * m * nsv,  # dO, v, I exp(-G), p exp(G) -> dv, slices of dI^v
        "bwd_dk_dIk_pair_rev": 3 * w.d_k * e + 8 * m + 4 * m * nsk,  # q, k, I exp(-G), dz exp(G) -> dk, slices of dI^k
        "gate_grad": 4 * m * (7 + nsk + nsv),   # u, gate, G, partials -> dgate; carry pass reads gate, r/w dgate
        # fused chunk kernels: the slot rows between the passes stay on chip
        "fused_fwd": e * (2 * w.d_k + 2 * w.d_v) + 12 * m,           # q, k, v, I exp(-G), G -> o, o'
        "fused_bwd": e * (2 * w.d_k + 2 * w.d_v) + 24 * m,           # dO, v, k, I exp(-G), G, o' -> dq, u, p exp(G), dz exp(G)
    }
    return R * table[label]


def kernel_function(label: str) -> str:
    """The kernel that serves a timing label: the four value_side scans of a step are launches
    of one kernel, and so are the four key_side scans."""
    if label.startswith("fused"):
        return "fused_pair_kernel"
    if "pair_rev" in label:
        return "rev_pair_kernel"
    if "key_side" in label:
        return "key_side_lean_kernel"
    if "value_side" in label:
        return "value_side_lean_kernel"
    return label


def kernel_algorithmic_flops(fn: str, w: W.Workload, d: int) -> float:
    """Dense flops of one launch of a chunk scan at C = 128 per token-head row, every product
    counted once (not per head-dimension slice, not per high/low operand part): the C x C
    slot-space or head-space product, the intra-chunk product, the inter-chunk product and
    the state update."""
    C, m = 128, w.m
    per_row = 2 * C * (m + d) + 4 * m * d      # (the same count for either primitive)
    if fn == "fused_pair_kernel":
        per_row *= 2                           # a value_side and a key_side scan
    if fn == "rev_pair_kernel":
        per_row = 4 * C * (m + d) + 6 * m * d  # ... that share the state update
    return float(per_row) * w.B * w.T * w.H


def step_flops(w: W.Workload) -> float:
    """Chunkwise forward flops per token-head at C = 128 (causal half counted),
    F = 4m(dk+dv) + C(dk+dv) + 2Cm, and 3.5x that for forward + backward."""
    C = 128
    f = 4 * w.m * (w.d_k + w.d_v) + C * (w.d_k + w.d_v) + 2 * C * w.m
    return 3.5 * f * w.B * w.T * w.H


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,utilization.gpu,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.idx}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    if float(f[3]) < 50.0:      # keep samples taken under load only
                        continue
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for n, v in zip(names, f[5:9]):
                    if v.lower() == "active":
                        reasons.add(n)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ----------------------------------------------------------------------------- reference arm
def oracle_step(x, w, pairs, threads, act="softmax"):
    import oracle
    rng = (0, pairs)
    oracle.fwd(x["q"], x["k"], x["v"], x["gate"], bh_range=rng, threads=threads, act=act)
    oracle.bwd(x["q"], x["k"], x["v"], x["gate"], x["dO"], bh_range=rng, threads=threads, act=act)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    w = W.CONFIGS[WORKLOAD]
    x = W.make_inputs(w)
    threads = min(oracle.default_threads(), 16, w.B * w.H)
    pairs = threads
    for _ in range(args.warmup):
        oracle_step(x, w, pairs, threads, args.slot_act)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(x, w, pairs, threads, args.slot_act)
    dt = (time.perf_counter() - t0) / args.steps
    tokens = pairs * w.T / w.H          # a token counts once all H heads are done
    val = tokens / dt
    sample = (f"{pairs} of {w.B * w.H} (batch, head) pairs of the {WORKLOAD} workload per step, "
              f"forward + reverse sweep in fp64; tokens = pairs * T / H")
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic (seeded, bf16-rounded inputs)",
        "config": {"workload": WORKLOAD, "B": w.B, "T": w.T, "H": w.H, "d_k": w.d_k, "d_v": w.d_v,
                   "m": w.m, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- sharding
def rank_workload(rank: int, m: int = 0) -> W.Workload:
    """Weak scaling over batch: rank r runs its own batch of the workload (its own seed);
    (batch, head) pairs are independent recurrences, so no rank needs another's data.
    m (0 = the workload's own 64): another slot count on the same shape (the paper's ablation on the
    number of slots: 32, 64, 128)."""
    base = W.CONFIGS[WORKLOAD]
    return base.scaled(seed=base.seed + 1000 * rank, m=m or base.m)


def max_over_ranks(ms: float, world: int, device=None) -> float:
    """Slowest rank's time (all-reduce MAX; works on nccl and gloo groups)."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(world: int, tokens_per_rank: int, ms_per_step: float) -> float:
    return world * tokens_per_rank / (ms_per_step * 1e-3)


# ----------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    import __graft_entry__ as entry
    entry.build()
    import paper_2409_07146_b200 as gsa

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the GSA library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)

    w = rank_workload(rank, args.m)
    x = W.make_inputs(w)
    p = gsa.Params(w.B, w.T, w.H, w.d_k, w.d_v, w.m, io=w.io, slot_act=args.slot_act, tc_operands=args.tc_operands,
                   fuse=args.fuse)

    def host(a, bf16):
        t = torch.from_numpy(np.ascontiguousarray(a))
        if bf16:
            t = t.to(torch.bfloat16)
        return t.pin_memory()

    h_in = {n: host(x[n], n != "gate") for n in ("q", "k", "v", "gate", "dO")}
    d_in = {n: t.to(dev) for n, t in h_in.items()}
    io = torch.bfloat16
    o = torch.empty(w.B, w.T, w.H, w.d_v, dtype=io, device=dev)
    ok = torch.empty(w.B, w.T, w.H, w.m, dtype=torch.float32, device=dev)
    dq = torch.empty(w.B, w.T, w.H, w.d_k, dtype=io, device=dev)
    dk = torch.empty_like(dq)
    dv = torch.empty_like(o)
    dg = torch.empty_like(ok)
    ws_f = torch.empty(gsa.gsa_workspace_bytes(p, 0), dtype=torch.uint8, device=dev)
    ws_b = torch.empty(gsa.gsa_workspace_bytes(p, 1), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    h_out = {n: torch.empty(t.shape, dtype=t.dtype).pin_memory()
             for n, t in (("o", o), ("dq", dq), ("dk", dk), ("dv", dv), ("dgate", dg))}

    outs = {"o": o, "dq": dq, "dk": dk, "dv": dv, "dgate": dg}

    # the forward leaves the gate kernel's products (as it leaves the logits) for the backward of
    # the same step: memory for time, 50 MB at this shape; --recompute-gate times the plain pair
    gate_blk = None if args.recompute_gate else gsa.gate_block(p, dev)

    def step(src, dst=outs):
        gsa.gsa_fwd(p, src["q"], src["k"], src["v"], src["gate"], o=dst["o"], ok_save=ok, ws=ws_f,
                    dev_status=status, gate_save=gate_blk)
        gsa.gsa_bwd(p, src["q"], src["k"], src["v"], src["gate"], src["dO"], ok_saved=ok, dq=dst["dq"],
                    dk=dst["dk"], dv=dst["dv"], dgate=dst["dgate"], ws=ws_b, dev_status=status,
                    gate_saved=gate_blk)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        return max_over_ranks(float(e0.elapsed_time(e1)), world, dev)

    if args.profile_case:
        # bare steps for a profiler: no timing, no extras (the numbers of such a run are not
        # benchmark values)
        if args.profile_case == "decode":
            wd = W.CONFIGS["decode"]
            pdec = gsa.Params(wd.B, 1, wd.H, wd.d_k, wd.d_v, wd.m, io="bf16")
            sd = W.make_decode_states(wd)
            Ks, Vs = torch.from_numpy(sd["K"]).to(dev), torch.from_numpy(sd["V"]).to(dev)
            xd = W.make_decode_step_inputs(wd, 0)
            qd, kd, vd = (torch.from_numpy(xd[n]).to(dev).to(torch.bfloat16) for n in ("q", "k", "v"))
            gd = torch.from_numpy(xd["gate"]).to(dev)
            od = torch.empty(wd.B, wd.H, wd.d_v, dtype=torch.bfloat16, device=dev)
            for _ in range(args.warmup + args.steps):
                gsa.gsa_decode_step(pdec, qd, kd, vd, gd, Ks, Vs, o=od)
        elif args.profile_case == "fwd":
            for _ in range(args.warmup + args.steps):
                gsa.gsa_fwd(p, d_in["q"], d_in["k"], d_in["v"], d_in["gate"], o=o, ws=ws_f, dev_status=status)
        else:
            for _ in range(args.warmup + args.steps):
                step(d_in)
        torch.cuda.synchronize()
        if rank == 0:
            print(json.dumps({"profile_case": True, "steps": args.steps, "warmup": args.warmup}))
        return
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        step(d_in)
    # One step = 22 kernels on six streams: it is captured once into a CUDA graph and the timed
    # region replays that graph (the library calls are capture-safe: no allocation, no host
    # synchronisation).  --no-graph times the plain calls instead.
    run_step, launch_mode = (lambda: step(d_in)), "library calls, one step after the other"
    if not args.no_graph:
        try:
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step(d_in)
            graph.replay()
            torch.cuda.synchronize()
            run_step, launch_mode = graph.replay, "CUDA graph of one step (captured after warm-up), replayed"
        except Exception as exc:      # capture not available: time the plain calls
            launch_mode += f" (graph capture failed: {type(exc).__name__})"
            torch.cuda.synchronize()
    total_ms = timed(run_step, args.steps)
    # The timed region lasts a few milliseconds, shorter than nvidia-smi's sampling period and too short
    # for the power limiter to settle: keep the same steps running for at least 1.5 s more, timed with
    # CUDA events as well, so that the clock samples and the `sustained` figure describe the same load.
    sust_steps, sust_ms = 0, 0.0
    t_end = time.perf_counter() + 1.5
    while time.perf_counter() < t_end:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(100):
            run_step()
        e1.record()
        torch.cuda.synchronize()
        sust_ms += float(e0.elapsed_time(e1))
        sust_steps += 100
    sust_ms = max_over_ranks(sust_ms, world, dev)
    clocks = sampler.stop() if rank == 0 else {}
    if rank == 0:
        clocks["note"] = ("nvidia-smi samples (50 ms period, utilisation >= 50%) over warm-up, the timed steps and "
                          "the sustained loop of the same steps that follows them")
    ms_step = total_ms / args.steps
    value = aggregate_tokens_per_s(world, w.tokens, ms_step)
    if int(status.item()) != 0:
        raise SystemExit("a bounded device-side wait expired during the benchmark")
    if not bool(torch.isfinite(dq.float()).all()):
        raise SystemExit("non-finite gradients")

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region.
    # Every step copies its inputs from pinned host memory and its results back; as a training
    # loop would, the copies of neighbouring steps overlap the computation: inputs of step i+1
    # go up and results of step i-1 come down (two buffer sets, three streams) while step i runs.
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    s_comp = torch.cuda.current_stream(dev)
    d_in2 = [d_in, {n: torch.empty_like(t) for n, t in d_in.items()}]
    outs2 = [outs, {n: torch.empty_like(t) for n, t in outs.items()}]
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_comp = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def e2e_steps_run(nsteps):
        for i in range(nsteps):
            b2 = i & 1
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_comp[b2])          # step i-2 has read this input set
                for n in h_in:
                    d_in2[b2][n].copy_(h_in[n], non_blocking=True)
                ev_in[b2].record(s_in)
            s_comp.wait_event(ev_in[b2])
            if i >= 2:
                s_comp.wait_event(ev_out[b2])             # results of step i-2 have left this output set
            step(d_in2[b2], outs2[b2])
            ev_comp[b2].record(s_comp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_comp[b2])
                for n in h_out:
                    h_out[n].copy_(outs2[b2][n], non_blocking=True)
                ev_out[b2].record(s_out)
        s_comp.wait_event(ev_out[(nsteps - 1) & 1])       # the timed region ends when the last results are down
        if nsteps >= 2:
            s_comp.wait_event(ev_out[nsteps & 1])

    e2e_steps_run(2)
    e2e_steps = max(4, args.steps // 2)
    e2e_ms = timed(lambda: e2e_steps_run(e2e_steps), 1) / e2e_steps
    h2d = sum(t.numel() * t.element_size() for t in h_in.values())
    d2h = sum(t.numel() * t.element_size() for t in h_out.values())

    line = None
    if rank == 0:
        # ---- per-kernel durations (a second pass over the same steps, kernels bracketed by events)
        pk = peaks()
        reps = max(3, min(args.steps, 10))
        gsa.gsa_timing_begin(64 * reps)
        for _ in range(reps):
            step(d_in)
        recs = gsa.gsa_timing_end(64 * reps)
        per = {}
        for lab, ms in recs:
            per.setdefault(lab, []).append(ms)
        # kernels behind one label: gate_grad is three; every chunk pass is two (the lean and the
        # general variant of the kernel are both launched, each CTA runs in one of them)
        two = sum(len(v) for lab, v in per.items() if lab.endswith("_side") or lab.endswith("_side_rev"))
        # a fused label is the fused kernel plus the three kernels that serve the flagged pairs
        fusedl = sum(len(v) for lab, v in per.items() if lab.startswith("fused"))
        # a pair label is the pair kernel plus the two general kernels that serve the flagged pairs
        pairl = sum(len(v) for lab, v in per.items() if "pair_rev" in lab)
        launches = (len(recs) + 2 * len(per.get("gate_grad", [])) + two + 3 * fusedl + 2 * pairl) // reps
        kernels = []
        tot = sum(sum(v) for v in per.values())
        for lab, v in per.items():
            avg = sum(v) / len(v)
            by = kernel_algorithmic_bytes(lab, w)
            kernels.append({"kernel": lab, "launches_per_step": len(v) // reps, "avg_ms": avg,
                            "share": sum(v) / tot, "alg_bytes": by,
                            "achieved_gbs": by / (avg * 1e-3) / 1e9,
                            "frac_of_hbm_peak": by / (avg * 1e-3) / 1e9 / pk["hbm_gbs"]})
        kernels.sort(key=lambda k: -k["share"])
        # the dominant kernel: the one with the largest total time over the step, all its launches
        # taken together (the four key_side scans are one kernel, the four value_side scans another)
        groups = {}
        for k_ in kernels:
            groups.setdefault(kernel_function(k_["kernel"]), []).append(k_)
        # (value_side and key_side take the same time to within a percent or two: among the kernels within 3%
        # of the largest total, the one furthest below its roofline is reported, so that the choice does not
        # flip between runs)
        share_of = {f_: sum(k_["share"] for k_ in ms_) for f_, ms_ in groups.items()}
        top = max(share_of.values())
        close = [f_ for f_ in groups if share_of[f_] >= 0.97 * top]
        fn = min(close, key=lambda f_: sum(k_["frac_of_hbm_peak"] * k_["launches_per_step"] for k_ in groups[f_]) /
                 sum(k_["launches_per_step"] for k_ in groups[f_]))
        members = groups[fn]
        n_l = sum(k_["launches_per_step"] for k_ in members)
        avg_ms = sum(k_["avg_ms"] * k_["launches_per_step"] for k_ in members) / n_l
        alg = sum(k_["alg_bytes"] * k_["launches_per_step"] for k_ in members) / n_l
        traf = [NCU_TRAFFIC.get(k_["kernel"]) for k_ in members]
        traffic = int(sum(traf) / len(traf)) if (all(t is not None for t in traf) and w.m == 64) else None
        # the bytes the same launch would move if the slot-sized rows between the passes stayed on chip
        # (the d-sized tensors only: v in, o out for key_side; q, k in for value_side)
        e_ = 2 if w.io == "bf16" else 4
        fused_bytes = w.B * w.T * w.H * (3 if fn == "rev_pair_kernel" else 2) * (w.d_v if fn.startswith("key") else w.d_k) * e_
        roofline = {"bound": "hbm", "kernel": fn, "labels": [k_["kernel"] for k_ in members],
                    "launches_per_step": n_l, "avg_launch_ms": avg_ms,
                    "achieved": alg / (avg_ms * 1e-3) / 1e9,
                    "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": alg / (avg_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                    "traffic": traffic, "traffic_source": ("profiles/step_kernels_train_1p3b_ncu_full.md (one ncu capture of "
                                                           "this workload; not measured in this run)") if traffic else None,
                    "frac_on_fused_bytes": fused_bytes / (avg_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                    "limiter": ("tile-copy throughput per SM: a CTA of a scan moves 2-3 MB through two shared-memory stages and one "
                                "SM sustains about 41 GB/s of TMA copies (knock-out builds: a value_side scan with nothing but its "
                                "copies and barrier hand-shakes takes 36.6 of its 50.8 us; removing the masks, the state update, the "
                                "read-out or any group of MMAs changes it by 1-3 us each); ncu: tensor pipe 58-67% active, DRAM at "
                                "32-50% of peak, 128 CTAs on 148 SMs"),
                    "peak_source": pk["source"],
                    "share_of_step": sum(k_["share"] for k_ in members)}
        if fn.endswith("_side_lean_kernel") or fn in ("fused_pair_kernel", "rev_pair_kernel"):
            d = w.d_v if fn.startswith("key") else w.d_k     # (d_k == d_v in the benchmark workload)
            fl = kernel_algorithmic_flops(fn, w, d)
            roofline["alg_tflops"] = fl / (avg_ms * 1e-3) / 1e12
            roofline["frac_of_bf16_peak"] = roofline["alg_tflops"] / pk["bf16_tflops"]
            roofline["note"] = ("flops per byte of the launch %.0f against a machine balance of %.0f: the HBM side of "
                                "the roofline bounds it; a third to a half of the tcgen05.mma of a chunk exist only for "
                                "the high/low operand pairs that keep every tensor within tolerance" % (fl / alg, pk["bf16_tflops"] * 1e12 / (pk["hbm_gbs"] * 1e9)))
        step_bytes = step_algorithmic_bytes(w)
        whole = {"alg_bytes_per_step": step_bytes,
                 "achieved_gbs": step_bytes / (ms_step * 1e-3) / 1e9,
                 "frac_of_hbm_peak": step_bytes / (ms_step * 1e-3) / 1e9 / pk["hbm_gbs"],
                 "tflops": step_flops(w) / (ms_step * 1e-3) / 1e12}

        # ---- decode step (the recurrent form), reported beside the training number
        decode = bench_decode(gsa, torch, dev, pk)
        others = [] if args.no_other_configs else bench_other_configs(gsa, torch, dev, pk, args)
        decode_loop = None if args.no_other_configs else bench_decode_loop(gsa, torch, dev)

        # ---- the oracle on the host cores, bounded sample
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            x0 = x
            threads = min(oracle.default_threads(), 16, w.B * w.H)
            pairs = min(w.B * w.H, 2 * threads)
            t0 = time.perf_counter()
            oracle_step(x0, w, pairs, threads, args.slot_act)
            dt = time.perf_counter() - t0
            cpu = {"value": pairs * w.T / w.H / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
                   "sample": f"{pairs} of {w.B * w.H} (batch, head) pairs of one {WORKLOAD} step, "
                             f"fp64 forward + reverse sweep, {dt:.1f} s wall"}

        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic (seeded N(0,1) q,k,v,dO; gate sigmoid(N(0,1))^(1/8))",
            "config": {"workload": WORKLOAD, "B": w.B, "T": w.T, "H": w.H, "d_k": w.d_k,
                       "d_v": w.d_v, "m": w.m, "io": w.io, "chunk": gsa.gsa_chunk_size(p),
                       "step": ("gsa_fwd (logits saved) + gsa_bwd" if args.recompute_gate else
                                "gsa_fwd_save_gate (logits and the gate kernel's products saved) + gsa_bwd_saved_gate"),
                       "slot_act": args.slot_act, "tc_operands": args.tc_operands,
                       "fused_slot_softmax": bool(args.fuse),
                       "launch": launch_mode,
                       "l2": "inputs larger than L2 (1.1 GB touched per step vs 126 MB)",
                       "parallelism": f"dp{world} over batch, no collective"},
            "clocks": clocks,
            "sustained": {"ms_per_step": sust_ms / sust_steps, "tokens_per_s": aggregate_tokens_per_s(world, w.tokens, sust_ms / sust_steps),
                          "steps": sust_steps, "seconds": sust_ms * 1e-3, "sm_mhz_median": clocks.get("sm_mhz"),
                          "ms_x_mhz": (sust_ms / sust_steps) * clocks["sm_mhz"] if clocks.get("sm_mhz") else None,
                          "note": "the same step replayed back to back for >= 1.5 s (power-capped clocks), CUDA events"},
            "e2e": {"value": world * w.tokens / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
                    "overlap": "every step copies its inputs up and its results down; copies of "
                               "neighbouring steps overlap the computation (two buffer sets, three streams)"},
            "gpu_launches": launches * args.steps,
            "gpu_launches_per_step": launches,
            "roofline": roofline,
            "whole_step": whole,
            "kernels": kernels,
            "decode": decode,
            "decode_loop": decode_loop,
            "configs": others,
            "cpu_baseline": cpu,
        }
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line), flush=True)


def run_seq_sharded(args):
    """--shard seq: every rank holds one T-shard of the same sequences (rank r: tokens [r T, (r+1) T) of a
    sequence of N T tokens), the shards' end memories are exchanged by one all-gather per direction
    (NCCL over NVLink; into local memory), everything else is the local step.  Weak scaling in T."""
    import torch
    import torch.distributed as dist
    import __graft_entry__ as entry
    entry.build()
    import paper_2409_07146_b200 as gsa
    from paper_2409_07146_b200 import seqshard

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the GSA library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    w = rank_workload(rank, args.m)          # (its own seed per rank: a different stretch of the long sequence)
    x = W.make_inputs(w)
    p = gsa.Params(w.B, w.T, w.H, w.d_k, w.d_v, w.m, io=w.io)
    xs = {n: torch.from_numpy(x[n]).to(dev).to(torch.bfloat16) for n in ("q", "k", "v")}
    xs["gate"] = torch.from_numpy(x["gate"]).to(dev)
    dO = torch.from_numpy(x["dO"]).to(dev).to(torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    eng = seqshard.CudaEngine(p, dev_status=status)
    gather = seqshard.dist_gather if world > 1 else (lambda t: t.unsqueeze(0).contiguous())

    def step():
        o, saved = seqshard.sharded_forward(eng, gather, rank, xs, w.d_k, w.d_v)
        return seqshard.sharded_backward(eng, gather, rank, xs, dO, saved, w.d_k, w.d_v)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms = max_over_ranks(float(e0.elapsed_time(e1)), world, dev) / args.steps
    clocks = sampler.stop() if rank == 0 else {}
    if int(status.item()) != 0:
        raise SystemExit("a bounded device-side wait expired during the benchmark")
    if rank == 0:
        exch = 4 * w.B * w.H * w.m * (w.d_k + w.d_v + 1) * 2      # forward and backward all-gather payload per rank
        print(json.dumps({
            "metric": METRIC, "value": aggregate_tokens_per_s(world, w.tokens, ms), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic (seeded)",
            "config": {"workload": WORKLOAD, "B": w.B, "T_per_rank": w.T, "T_total": w.T * world, "H": w.H, "d_k": w.d_k,
                       "d_v": w.d_v, "m": w.m, "parallelism": f"sp{world}: sequence sharded over T, one all-gather of shard "
                       "memories per direction, the backward's local step run twice",
                       "launch": "plain library calls", "l2": "inputs larger than L2",
                       "exchange_bytes_per_rank_per_step": exch,
                       "note": "N > 1 is unmeasured on hardware in this build (single-GPU runs only)" if world == 1 else None},
            "clocks": clocks, "gpu_launches": None}), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def forward_algorithmic_bytes(w: W.Workload) -> int:
    """q, k, v, gate in; o out (no saved logits)."""
    e = 2 if w.io == "bf16" else 4
    return w.B * w.T * w.H * (e * (2 * w.d_k + 2 * w.d_v) + 4 * w.m)


def bench_other_configs(gsa, torch, dev, pk, args):
    """The other configurations, outside the headline region: plain library calls, CUDA events,
    whole-call time and the fraction of the HBM bound on the bytes every tensor must cross HBM once."""
    out = []
    plan = [("train_2p7b", True, 10), ("t2r_7b", True, 10), ("long_keep", False, 10), ("long_forget", False, 5),
            ("tiny_f32", False, 50)]
    for name, with_bwd, reps in plan:
        w = W.CONFIGS[name]
        x = W.make_inputs(w)
        p = gsa.Params(w.B, w.T, w.H, w.d_k, w.d_v, w.m, io=w.io, fuse=args.fuse)

        def dev_t(a, io_typed):
            t = torch.from_numpy(np.ascontiguousarray(a)).to(dev)
            return t.to(torch.bfloat16) if (io_typed and w.io == "bf16") else t

        q, k, v = (dev_t(x[n], True) for n in ("q", "k", "v"))
        gate = dev_t(x["gate"], False)
        K0 = dev_t(x["K0"], False) if "K0" in x else None
        V0 = dev_t(x["V0"], False) if "V0" in x else None
        dO = dev_t(x["dO"], True) if with_bwd else None
        o = torch.empty(w.B, w.T, w.H, w.d_v, dtype=p.io_dtype, device=dev)
        ok = torch.empty(w.B, w.T, w.H, w.m, device=dev) if with_bwd else None
        KT = torch.empty(w.B, w.H, w.m, w.d_k, device=dev) if K0 is not None else None
        VT = torch.empty(w.B, w.H, w.m, w.d_v, device=dev) if V0 is not None else None
        ws_f = torch.empty(max(gsa.gsa_workspace_bytes(p, 0), 256), dtype=torch.uint8, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        blk = gsa.gate_block(p, dev) if with_bwd else None
        if with_bwd:
            ws_b = torch.empty(gsa.gsa_workspace_bytes(p, 1), dtype=torch.uint8, device=dev)
            dq, dk, dv, dg = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v), torch.empty_like(gate)

        def fwd():
            gsa.gsa_fwd(p, q, k, v, gate, K0, V0, o=o, ok_save=ok, KT=KT, VT=VT, ws=ws_f, dev_status=status, gate_save=blk)

        def bwd():
            gsa.gsa_bwd(p, q, k, v, gate, dO, K0, V0, ok_saved=ok, dq=dq, dk=dk, dv=dv, dgate=dg, ws=ws_b,
                        dev_status=status, gate_saved=blk)

        def time_ms(fn):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return float(e0.elapsed_time(e1)) / reps

        f_ms = time_ms(fwd)
        rec = {"workload": name, "B": w.B, "T": w.T, "H": w.H, "d": w.d_k, "m": w.m, "io": w.io,
               "fwd_ms": f_ms, "fwd_tokens_per_s": w.tokens / (f_ms * 1e-3)}
        by = forward_algorithmic_bytes(w)
        if with_bwd:
            b_ms = time_ms(bwd)
            by = step_algorithmic_bytes(w)
            rec.update(bwd_ms=b_ms, step_ms=f_ms + b_ms, step_tokens_per_s=w.tokens / ((f_ms + b_ms) * 1e-3))
        t_ms = rec.get("step_ms", f_ms)
        rec.update(alg_bytes=by, frac_of_hbm_peak=by / (t_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                   launch="plain library calls" + (", gate kernel's products saved for the backward" if with_bwd else ""))
        if name == "tiny_f32":
            rec["note"] = "latency of one call (launch-bound); the fraction of the HBM bound means nothing at this size"
        if int(status.item()) != 0:
            rec["error"] = "a bounded device-side wait expired"
        out.append(rec)
        del q, k, v, gate, o
        torch.cuda.empty_cache()
    return out


def bench_decode(gsa, torch, dev, pk):
    """gsa_decode_step on the batched-decoding workload (256 sequences x 32 heads, d=128,
    m=64, fp32 memories): achieved HBM GB/s on the bytes one step must move."""
    w = W.CONFIGS["decode"]
    p = gsa.Params(w.B, 1, w.H, w.d_k, w.d_v, w.m, io="bf16")
    st = W.make_decode_states(w)
    Ks = torch.from_numpy(st["K"]).to(dev)
    Vs = torch.from_numpy(st["V"]).to(dev)
    xs = W.make_decode_step_inputs(w, 0)
    q, k, v = (torch.from_numpy(xs[n]).to(dev).to(torch.bfloat16) for n in ("q", "k", "v"))
    gate = torch.from_numpy(xs["gate"]).to(dev)
    o = torch.empty(w.B, w.H, w.d_v, dtype=torch.bfloat16, device=dev)
    for _ in range(10):
        gsa.gsa_decode_step(p, q, k, v, gate, Ks, Vs, o=o)
    torch.cuda.synchronize()
    steps = 100
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        gsa.gsa_decode_step(p, q, k, v, gate, Ks, Vs, o=o)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    pairs = w.B * w.H
    by = pairs * (2 * 4 * w.m * (w.d_k + w.d_v) + 2 * (2 * w.d_k + 2 * w.d_v) + 4 * w.m)
    return {"workload": "decode (256 seqs x 32 heads, d=128, m=64)", "us_per_step": ms * 1e3,
            "tokens_per_s": w.B / (ms * 1e-3), "alg_bytes_per_step": by,
            "achieved_gbs": by / (ms * 1e-3) / 1e9,
            "frac_of_hbm_peak": by / (ms * 1e-3) / 1e9 / pk["hbm_gbs"],
            "note": "states (1.07 GB read+write per step) exceed L2"}


def free_port() -> int:
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def launcher_command(n: int, argv):
    """The command that runs this script as n ranks on one node (one rank per GPU, rendezvous on the
    loopback address)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__), *argv]


def bench_decode_loop(gsa, torch, dev):
    """Token-by-token decoding through the GSA layers of the whole 1.3B model: 24 layers, each one
    gsa_decode_step on its own memories (one sequence, 4 heads of width 512, 64 slots), the 24 steps of a
    token captured once as a CUDA graph and replayed per token.  Only the GSA layers: no projections,
    no GLU, no sampling.  The paper's 211 s for 16K tokens is the whole model on one H800 -- context."""
    w = W.CONFIGS["decode_1p3b"]
    layers = 24
    p = gsa.Params(w.B, 1, w.H, w.d_k, w.d_v, w.m, io="bf16")
    st = W.make_decode_states(w)
    Ks = [torch.from_numpy(st["K"]).to(dev).clone() for _ in range(layers)]
    Vs = [torch.from_numpy(st["V"]).to(dev).clone() for _ in range(layers)]
    xs = W.make_decode_step_inputs(w, 0)
    q, k, v = (torch.from_numpy(xs[n]).to(dev).to(torch.bfloat16) for n in ("q", "k", "v"))
    gate = torch.from_numpy(xs["gate"]).to(dev)
    o = torch.empty(w.B, w.H, w.d_v, dtype=torch.bfloat16, device=dev)

    def token():
        for l in range(layers):
            gsa.gsa_decode_step(p, q, k, v, gate, Ks[l], Vs[l], o=o)

    for _ in range(3):
        token()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        token()
    tokens = 2048
    for _ in range(20):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(tokens):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    us = float(e0.elapsed_time(e1)) * 1e3 / tokens
    state_bytes = layers * w.H * w.m * (w.d_k + w.d_v) * 4
    return {"workload": "decode_1p3b: 24 GSA layers x (1 sequence, 4 heads, d=512, m=64), one token at a time",
            "us_per_token": us, "tokens_per_s": 1e6 / us, "seconds_for_16k_tokens": us * 16384 * 1e-6,
            "state_bytes": state_bytes, "achieved_gbs": 2 * state_bytes / (us * 1e-6) / 1e9,
            "launch": "CUDA graph of the 24 decode steps of a token, replayed per token",
            "paper_context": "whole 1.3B model, 1 x H800, 2K prefix + 16K generated: 211.0 s (another metric: the "
                             "model's projections, GLU layers and sampling are not in this figure)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--recompute-gate", action="store_true",
                    help="plain gsa_fwd + gsa_bwd: the backward runs the gate kernel again instead of reading the "
                         "forward's saved block")
    ap.add_argument("--tc-operands", default="paired", choices=["paired", "single"],
                    help="derived operands of the tensor-core kernels as bf16 high/low pairs (default) or as one "
                         "bf16 value")
    ap.add_argument("--slot-act", default="softmax", choices=["softmax", "none", "relu", "swish", "relu2"],
                    help="the non-linearity between the two passes: the paper's softmax (the headline "
                         "workload) or one of the replacements of its ablation")
    ap.add_argument("--shard", default="batch", choices=["batch", "seq"],
                    help="how N ranks share the work: batch (the default: every rank its own batch, no collective) or "
                         "seq (every rank a T-shard of the same sequences, one all-gather of shard memories)")
    ap.add_argument("--m", type=int, default=0, choices=[0, 32, 64, 128],
                    help="slot count on the benchmark shape (default: the workload's 64); 32 runs on the tensor-core "
                         "kernels' 64-slot tiles, 128 on the fp32 CUDA-core kernels")
    ap.add_argument("--fuse", action="store_true",
                    help="the fused chunk kernel (pass 1 -> slot softmax -> pass 2 in one kernel, and its backward "
                         "twin) instead of the separate kernels; slower as measured, not the default")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the list of the other configurations (t2r_7b, long_keep, long_forget, tiny_f32)")
    ap.add_argument("--no-graph", action="store_true", help="time plain library calls instead of a CUDA graph replay")
    ap.add_argument("--profile-case", nargs="?", const="step", default=None, choices=["step", "fwd", "decode"],
                    help="run warmup + steps of one case bare (for ncu; prints no benchmark line): step = the "
                         "benchmark's forward + backward, fwd = the forward alone without saved logits (with --fuse: "
                         "the fused kernel), decode = gsa_decode_step on the decode workload")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain process: start the N ranks of one node here (what a torchrun command line does)
        raise SystemExit(subprocess.call(launcher_command(args.gpus, sys.argv[1:])))
    if args.impl == "reference":
        run_reference(args)
    elif args.shard == "seq":
        run_seq_sharded(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
