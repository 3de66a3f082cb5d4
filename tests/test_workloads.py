"""The seeded input generators: determinism, value recipe, bf16 rounding."""
import numpy as np
import torch

import gsa_workloads as W


def test_bf16_rounding_matches_torch_rne():
    x = np.random.default_rng(0).standard_normal(100000).astype(np.float32) * 37.0
    mine = W.round_to_bf16(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(mine, ref)
    bits = W.bf16_bits(mine)
    back = torch.from_numpy(bits.copy()).view(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(back, mine)


def test_streams_are_seeded_and_independent():
    w = W.CONFIGS["tiny_f32"]
    a, b = W.make_inputs(w), W.make_inputs(w)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])
    # dropping optional tensors does not change the others
    c = W.make_inputs(w.scaled(with_dO=False, init_state=True))
    np.testing.assert_array_equal(a["q"], c["q"])
    np.testing.assert_array_equal(a["gate"], c["gate"])
    assert "dO" not in c and c["K0"].shape == (1, 2, 32, 64)
    d = W.make_inputs(w.scaled(seed=5))
    assert np.abs(d["q"] - a["q"]).max() > 0.1


def test_value_recipe():
    w = W.CONFIGS["t2r_7b"].scaled(B=1, T=512)
    x = W.make_inputs(w)
    assert x["q"].shape == (1, 512, 32, 128) and x["gate"].shape == (1, 512, 32, 64)
    assert abs(x["q"].std() * 128 ** 0.5 - 1) < 0.02
    assert abs(x["v"].std() - 1) < 0.02
    # per-channel log-normal key scale: channel stds vary by about exp(0.5 N(0,1))
    ch = np.log(x["k"].std(axis=(0, 1)))
    assert 0.35 < ch.std() < 0.65
    g = x["gate"]
    assert g.dtype == np.float32 and g.min() > 0.3 and g.max() < 1.0
    # median of sigmoid(N(0,1))**(1/8) is 0.5**(1/8)
    assert abs(np.median(g) - 0.5 ** 0.125) < 0.01
    # bf16 workloads hold exactly representable values
    np.testing.assert_array_equal(W.round_to_bf16(x["k"]), x["k"])
    f = W.make_inputs(W.CONFIGS["long_forget"].scaled(T=256))
    assert abs(np.median(f["gate"]) - 1 / (1 + np.exp(2.0))) < 0.02


def test_decode_inputs():
    w = W.CONFIGS["decode"].scaled(B=4)
    s = W.make_decode_states(w)
    assert s["K"].shape == (4, 32, 64, 128) and abs(s["K"].std() - 0.1) < 0.005
    a, b = W.make_decode_step_inputs(w, 3), W.make_decode_step_inputs(w, 4)
    assert a["q"].shape == (4, 32, 128) and np.abs(a["q"] - b["q"]).max() > 0.01
    np.testing.assert_array_equal(a["v"], W.make_decode_step_inputs(w, 3)["v"])
