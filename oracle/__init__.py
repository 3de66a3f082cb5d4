"""Sequential fp64 CPU oracle for Gated Slot Attention -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA library and its Python binding never do, and the two
share no code.

``fwd`` / ``bwd`` / ``decode_step`` marshal numpy arrays into the plain C
recurrence of ``gsa_oracle.c`` (Eq. 6 of arXiv 2409.07146, evaluated one token
at a time in double precision) and spread the independent (batch, head) pairs
over host threads.  ``unrolled.py`` and ``chunkwise.py`` hold second and third
statements of the same function that the CPU tests use to pin this one.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gsa_oracle.c")
_SO = os.path.join(_HERE, "libgsa_oracle.so")
_lock = threading.Lock()
_lib = None

_D = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no CUDA involved) and return the .so path."""
    with _lock:
        if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
            tmp = _SO + ".tmp.%d" % os.getpid()
            subprocess.check_call(
                ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i, d = ctypes.c_int, ctypes.c_double
        lib.gsa_oracle_fwd.argtypes = [i] * 8 + [d] + [_D] * 10 + [i, i]
        lib.gsa_oracle_fwd.restype = i
        lib.gsa_oracle_decode_step.argtypes = [i] * 7 + [d] + [_D] * 7 + [i, i]
        lib.gsa_oracle_decode_step.restype = i
        lib.gsa_oracle_bwd.argtypes = [i] * 8 + [d] + [_D] * 15 + [i, i]
        lib.gsa_oracle_bwd.restype = i
        _lib = lib
    return _lib


def _f64(x, shape=None):
    if x is None:
        return None
    a = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {shape}, got {a.shape}")
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(_D)


def default_threads() -> int:
    return max(1, len(os.sched_getaffinity(0)))


def _run_split(fn, n_items: int, threads: int | None):
    """Call fn(begin, end) over a partition of range(n_items) on host threads."""
    nt = max(1, min(threads or default_threads(), n_items))
    bounds = [(n_items * j // nt, n_items * (j + 1) // nt) for j in range(nt)]
    if nt == 1:
        rcs = [fn(*bounds[0])]
    else:
        with ThreadPoolExecutor(nt) as ex:
            rcs = list(ex.map(lambda be: fn(*be), bounds))
    if any(rc != 0 for rc in rcs):
        raise RuntimeError(f"oracle returned {rcs}")
    return nt


# The non-linearity between the two passes: Eq. 6's softmax over the slots, or one of the
# element-wise replacements of the paper's ablation (Table "ablations": no softmax, Swish, ReLU,
# squared ReLU).
ACTS = {"softmax": 0, "none": 1, "relu": 2, "swish": 3, "relu2": 4}


def gate_from_logits(x, tau):
    """The layer's damped forget gate (Sec. 3.3): a = sigmoid(x)^(1/tau), and da/dx =
    a (1 - sigmoid(x)) / tau.  Returns (a, da_dx) in float64."""
    x = np.asarray(x, dtype=np.float64)
    sig = 1.0 / (1.0 + np.exp(-x))
    a = np.power(sig, 1.0 / float(tau))
    return a, a * (1.0 - sig) / float(tau)


def fwd(q, k, v, gate, *, gate_is_log=False, scale=1.0, K0=None, V0=None,
        bh_range=None, threads=None, gate_is_logits=False, tau=8.0, act="softmax"):
    """Eq. 6 over whole sequences.

    q,k [B,T,H,d_k]; v [B,T,H,d_v]; gate [B,T,H,m] (a, or log a when
    gate_is_log).  Returns dict(o, ok, KT, VT): outputs, scaled pre-softmax slot
    logits [B,T,H,m], final memories [B,H,m,d].  ``bh_range=(lo, hi)`` restricts
    the work to those flattened (b,h) pairs; the other entries stay zero.
    With gate_is_logits the gate tensor holds x and a = sigmoid(x)^(1/tau) (Sec. 3.3).
    ``act`` (a key of ACTS) replaces the softmax over the slots.
    """
    lib = _load()
    if gate_is_logits:
        gate, gate_is_log = gate_from_logits(gate, tau)[0], False
    q = _f64(q); B, T, H, dk = q.shape
    k = _f64(k, (B, T, H, dk))
    v = _f64(v); dv = v.shape[-1]
    gate = _f64(gate); m = gate.shape[-1]
    K0 = _f64(K0, (B, H, m, dk)) if K0 is not None else None
    V0 = _f64(V0, (B, H, m, dv)) if V0 is not None else None
    o = np.zeros((B, T, H, dv)); ok = np.zeros((B, T, H, m))
    KT = np.zeros((B, H, m, dk)); VT = np.zeros((B, H, m, dv))
    lo, hi = bh_range if bh_range is not None else (0, B * H)

    def run(b0, b1):
        return lib.gsa_oracle_fwd(B, T, H, dk, dv, m, int(gate_is_log), ACTS[act], float(scale),
                                  _p(q), _p(k), _p(v), _p(gate), _p(K0), _p(V0),
                                  _p(o), _p(ok), _p(KT), _p(VT), lo + b0, lo + b1)

    nt = _run_split(run, hi - lo, threads)
    return dict(o=o, ok=ok, KT=KT, VT=VT, threads=nt)


def bwd(q, k, v, gate, dO, *, gate_is_log=False, scale=1.0, K0=None, V0=None,
        dKT=None, dVT=None, bh_range=None, threads=None, gate_is_logits=False, tau=8.0,
        act="softmax"):
    """Reverse sweep of Eq. 6.  Returns dict(dq, dk, dv, dgate, dK0, dV0);
    dgate is the total derivative w.r.t. the gate tensor as passed (with gate_is_logits:
    w.r.t. x, through a = sigmoid(x)^(1/tau))."""
    if gate_is_logits:
        a, da_dx = gate_from_logits(gate, tau)
        r = bwd(q, k, v, a, dO, gate_is_log=False, scale=scale, K0=K0, V0=V0, dKT=dKT, dVT=dVT,
                bh_range=bh_range, threads=threads, act=act)
        r["dgate"] = r["dgate"] * da_dx
        return r
    lib = _load()
    q = _f64(q); B, T, H, dk = q.shape
    k = _f64(k, (B, T, H, dk))
    v = _f64(v); dv = v.shape[-1]
    gate = _f64(gate); m = gate.shape[-1]
    dO = _f64(dO, (B, T, H, dv))
    K0 = _f64(K0, (B, H, m, dk)) if K0 is not None else None
    V0 = _f64(V0, (B, H, m, dv)) if V0 is not None else None
    dKT = _f64(dKT, (B, H, m, dk)) if dKT is not None else None
    dVT = _f64(dVT, (B, H, m, dv)) if dVT is not None else None
    dq = np.zeros_like(q); dk_ = np.zeros_like(k); dv_ = np.zeros_like(v)
    dgate = np.zeros_like(gate)
    dK0 = np.zeros((B, H, m, dk)); dV0 = np.zeros((B, H, m, dv))
    lo, hi = bh_range if bh_range is not None else (0, B * H)

    def run(b0, b1):
        return lib.gsa_oracle_bwd(B, T, H, dk, dv, m, int(gate_is_log), ACTS[act], float(scale),
                                  _p(q), _p(k), _p(v), _p(gate), _p(K0), _p(V0),
                                  _p(dO), _p(dKT), _p(dVT), _p(dq), _p(dk_), _p(dv_),
                                  _p(dgate), _p(dK0), _p(dV0), lo + b0, lo + b1)

    nt = _run_split(run, hi - lo, threads)
    return dict(dq=dq, dk=dk_, dv=dv_, dgate=dgate, dK0=dK0, dV0=dV0, threads=nt)


def decode_step(q, k, v, gate, Kstate, Vstate, *, gate_is_log=False, scale=1.0,
                threads=None, gate_is_logits=False, tau=8.0, act="softmax"):
    """One recurrent step of Eq. 6 for S sequences; q,k [S,H,d_k], v [S,H,d_v],
    gate [S,H,m]; Kstate/Vstate [S,H,m,d] float64 C-contiguous arrays updated IN
    PLACE.  Returns o [S,H,d_v]."""
    lib = _load()
    if gate_is_logits:
        gate, gate_is_log = gate_from_logits(gate, tau)[0], False
    q = _f64(q); S, H, dk = q.shape
    k = _f64(k, (S, H, dk))
    v = _f64(v); dv = v.shape[-1]
    gate = _f64(gate); m = gate.shape[-1]
    for st, d in ((Kstate, dk), (Vstate, dv)):
        if not (isinstance(st, np.ndarray) and st.dtype == np.float64
                and st.flags.c_contiguous and st.shape == (S, H, m, d)):
            raise ValueError("states must be C-contiguous float64 [S,H,m,d] arrays")
    o = np.zeros((S, H, dv))

    def run(s0, s1):
        return lib.gsa_oracle_decode_step(S, H, dk, dv, m, int(gate_is_log), ACTS[act], float(scale),
                                          _p(q), _p(k), _p(v), _p(gate), _p(Kstate),
                                          _p(Vstate), _p(o), s0, s1)

    _run_split(run, S * H, threads)
    return o


def fwd_packed(q, k, v, gate, cu_seqlens, **kw):
    """Variable-length batches packed along T: every batch row holds the sequences
    [cu_seqlens[i], cu_seqlens[i+1]) back to back, each an independent recurrence of Eq. 6 from
    empty memories (K0 / V0, if given, enter the first one).  Plain definition: one `fwd` call per
    sequence on its slice.  Returns dict(o, ok, KT, VT) with KT / VT those of the last sequence."""
    cu = [int(c) for c in cu_seqlens]
    K0, V0 = kw.pop("K0", None), kw.pop("V0", None)
    parts = []
    for i in range(len(cu) - 1):
        sl = slice(cu[i], cu[i + 1])
        parts.append(fwd(q[:, sl], k[:, sl], v[:, sl], gate[:, sl], K0=K0 if i == 0 else None,
                         V0=V0 if i == 0 else None, **kw))
    return dict(o=np.concatenate([p["o"] for p in parts], axis=1), ok=np.concatenate([p["ok"] for p in parts], axis=1),
                KT=parts[-1]["KT"], VT=parts[-1]["VT"])


def bwd_packed(q, k, v, gate, dO, cu_seqlens, **kw):
    """Gradients of `fwd_packed`: one `bwd` call per sequence (dKT / dVT, if given, act on the last
    sequence's final memories; dK0 / dV0 are those of the first sequence's initial memories)."""
    cu = [int(c) for c in cu_seqlens]
    K0, V0, dKT, dVT = (kw.pop(n, None) for n in ("K0", "V0", "dKT", "dVT"))
    n = len(cu) - 1
    parts = []
    for i in range(n):
        sl = slice(cu[i], cu[i + 1])
        parts.append(bwd(q[:, sl], k[:, sl], v[:, sl], gate[:, sl], dO[:, sl], K0=K0 if i == 0 else None,
                         V0=V0 if i == 0 else None, dKT=dKT if i == n - 1 else None, dVT=dVT if i == n - 1 else None, **kw))
    out = {name: np.concatenate([p[name] for p in parts], axis=1) for name in ("dq", "dk", "dv", "dgate")}
    out["dK0"], out["dV0"] = parts[0]["dK0"], parts[0]["dV0"]
    return out
