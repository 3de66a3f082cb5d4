"""Helpers shared by the GPU parity tests: moving seeded numpy inputs to the device,
the error metric, and running the fp64 oracle on the values the GPU saw."""
import numpy as np
import torch

import oracle

TOL = {"f32": 1e-4, "bf16": 2e-2}   # max |x - ref| / rms(ref), outputs and gradients


def to_dev(x, io=None):
    """numpy float32 array -> CUDA tensor; io in {"f32","bf16"} picks the element type of
    q/k/v-like tensors (values are already representable), None keeps float32."""
    if x is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda()
    if io == "bf16":
        t = t.to(torch.bfloat16)
    return t.contiguous()


def to_np(t):
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


BF16_IO = {"o", "dq", "dk", "dv"}   # tensors stored in the io type (bf16 when io == "bf16")

# Bounds of the tensor-core path at the size of the benchmark configurations, per tensor, on
# max|err| / rms(ref):  ("plain", x) = no allowance;  ("bf16out", x) = after the half-ulp of the
# tensor's bfloat16 storage (bf16_half_ulp).  The fp32 outputs (logits, final memories, gate
# gradient) measure 1e-4, o and dv 1.4-1.8e-2 (the rounding of their bfloat16 storage), all on the
# plain metric.  dq and dk are stored as bfloat16 and heavy-tailed (max|ref| / rms = 10-11 at
# train_1p3b, 39 for dq at t2r_7b, where key channels carry outliers): the half-ulp of the output
# format alone (2^-9 to 2^-8 of |ref|) is then 2.6-6.8e-2 of the rms, above the stated 2e-2 on the
# plain metric, so these two meet the bound only after that half-ulp is taken off (what is left is
# 1e-4 and less).  Their plain figures are held under the ceilings of TC_PLAIN_CEILING, and every
# bfloat16-stored tensor is checked against the oracle's value rounded to bfloat16
# (bf16_storage_check).
TC_CONFIG_BOUNDS = {
    "o": ("plain", 2e-2), "ok": ("plain", 2e-2), "KT": ("plain", 2e-2),
    "VT": ("plain", 2e-2), "dv": ("plain", 2e-2), "dq": ("bf16out", 2e-2),
    "dk": ("bf16out", 2e-2), "dgate": ("plain", 2e-2),
}
# plain max|err| / rms of dq and dk as measured (train_1p3b 2.6e-2 / 3.3e-2, t2r_7b 6.8e-2 / 1.9e-2)
# plus 10%: the half-ulp of bfloat16 at the largest elements
TC_PLAIN_CEILING = {
    ("train_1p3b", "dq"): 2.9e-2, ("train_1p3b", "dk"): 3.7e-2,
    ("t2r_7b", "dq"): 7.5e-2, ("t2r_7b", "dk"): 2.1e-2,
}


def bf16_half_ulp(ref):
    """Half the spacing of bfloat16 numbers (8 significant bits) at |ref|: the largest error that
    rounding an exact result to bfloat16 can make.  Between 2^-9 |ref| and 2^-8 |ref|."""
    a = np.abs(np.asarray(ref, dtype=np.float64))
    e = np.floor(np.log2(np.maximum(a, 1e-300)))
    return np.where(a > 0, 2.0 ** (e - 8), 0.0)


def bf16_storage_check(x, ref):
    """Direct check of the reading that a bfloat16-stored result differs from the oracle by the
    rounding of its storage format and nothing else: every element of x must lie within one
    bfloat16 ulp (2^-7 of the binade) of the oracle value rounded to nearest-even bfloat16.  The
    ulp is taken at max(|ref|, 2e-2 rms(ref)): below that size an ulp is finer than the fp32
    arithmetic behind the result.  Returns (largest distance in such ulps, fraction of elements
    that are bit-equal to the rounded oracle value)."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rms = np.sqrt(np.mean(ref ** 2))
    a = np.abs(ref)
    e = np.floor(np.log2(np.maximum(a, 1e-300)))
    ulp = np.where(a > 0, 2.0 ** (e - 7), 0.0)
    rne = np.where(a > 0, np.rint(ref / np.where(ulp > 0, ulp, 1.0)) * ulp, 0.0)
    floor = max(2e-2 * rms, 1e-300)
    ulp_eff = 2.0 ** (np.floor(np.log2(np.maximum(a, floor))) - 7)
    worst = float((np.abs(x - rne) / ulp_eff).max())
    return worst, float(np.mean(x == rne))


def rel_err(x, ref, stored_bf16=False):
    """max |x - ref| / rms(ref): the normalisation used for every tolerance.

    For a tensor that the library stores as bfloat16, the half-ulp rounding of the result
    itself (bf16_half_ulp(ref) per element) is taken off first: with heavy-tailed gradients
    max|ref| / rms reaches 15-40, and the output format alone would then exceed the 2e-2
    bound however exact the arithmetic."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    diff = np.abs(x - ref)
    if stored_bf16:
        diff = np.maximum(diff - bf16_half_ulp(ref), 0.0)
    rms = np.sqrt(np.mean(ref ** 2))
    if rms == 0:
        return float(diff.max())
    return float(diff.max() / rms)


def rand_inputs(seed, B, T, H, dk, dv, m, io, init=False, final_grads=False, gate="tau8"):
    r = np.random.default_rng(seed)
    f = lambda *s: r.standard_normal(s).astype(np.float32)
    d = dict(q=f(B, T, H, dk) * np.float32(dk ** -0.5), k=f(B, T, H, dk), v=f(B, T, H, dv),
             dO=f(B, T, H, dv))
    x = r.standard_normal((B, T, H, m))
    sig = 1 / (1 + np.exp(-x))
    if gate == "tau8":
        a = sig ** 0.125
    elif gate == "strong":
        a = 1 / (1 + np.exp(-(x - 3.0)))
    elif gate == "mixed":        # some slots forget hard, some keep everything, exact 0 and 1
        a = sig ** 0.125
        a[..., 0] = 0.0
        a[..., 1] = 1.0
        a[..., 2] = 1 / (1 + np.exp(-(x[..., 2] - 4.0)))
    else:
        raise ValueError(gate)
    d["gate"] = a.astype(np.float32)
    if init:
        d["K0"] = f(B, H, m, dk) * np.float32(0.3)
        d["V0"] = f(B, H, m, dv) * np.float32(0.3)
    if final_grads:
        d["dKT"] = f(B, H, m, dk) * np.float32(0.3)
        d["dVT"] = f(B, H, m, dv) * np.float32(0.3)
    if io == "bf16":
        import gsa_workloads as W
        for n in ("q", "k", "v", "dO"):
            d[n] = W.round_to_bf16(d[n])
    return d
