"""The seeded input generator: deterministic, right shapes/dtypes/statistics."""
import numpy as np
import torch

import synth


def test_cases_cover_the_five_configurations():
    assert sorted(synth.CONFIGS) == [1, 2, 3, 4, 5]
    c3 = {c.name: (c.Cin, c.Cout) for c in synth.config_cases(3)}
    assert c3 == {"vitb_qkv": (768, 2304), "vitb_proj": (768, 768),
                  "vitb_fc1": (768, 3072), "vitb_fc2": (3072, 768)}
    for cases in synth.CONFIGS.values():
        for c in cases:
            assert c.H % c.k == 0 and c.W % c.k == 0
            assert max(c.ranks) <= c.k * c.k


def test_deterministic_and_distinct_streams():
    case = synth.config_cases(1)[0]
    a = synth.make_layer_inputs(case)
    b = synth.make_layer_inputs(case)
    for t, u in zip(a, b):
        assert torch.equal(t, u)
    x, gy, w = a
    assert x.shape == (2, 16, 16, 64) and gy.shape == (2, 16, 16, 64) and w.shape == (64, 64)
    assert x.dtype == torch.float32
    assert not torch.equal(x, gy)
    c = synth.make_layer_inputs(case, seed=synth.SEED + 1)
    assert not torch.equal(c[0], x)


def test_distributions():
    n = 200_000
    z = synth.make_tensor((n,), ("normal", 0.01), "f32", case_key=99).double().numpy()
    assert abs(z.mean()) < 2e-4 and abs(z.std() - 0.01) < 2e-4
    g = synth.make_tensor((n,), ("gelu_normal",), "f32", case_key=99).double().numpy()
    assert g.min() > -0.18 and abs(g.mean() - 0.2821) < 0.01     # E[GELU(z)] = 1/sqrt(4 pi)
    t = synth.make_tensor((n,), ("student_t4",), "f32", case_key=99).double().numpy()
    assert abs(t.var() - 2.0) < 0.3 and np.abs(t).max() > 8.0     # var = nu/(nu-2), heavy tail
    b = synth.make_tensor((64,), ("normal", 1.0), "bf16", case_key=99)
    assert b.dtype == torch.bfloat16
