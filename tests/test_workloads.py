"""The seeded input generator: determinism, routing validity and the stated shapes."""
import pytest
import numpy as np
import torch

from workloads import synth


def test_specs_match_stated_shapes():
    s = synth.SPECS
    assert s["c1"].shape == synth.Shape(8, 2, 256, 512) and s["c1"].ops == ((1, 48), (0, 16))
    assert s["c2"].shape == synth.Shape(256, 8, 3072, 1536) and s["c2"].ops == ((0, 128),)
    assert s["c3"].ops == ((1, 8192),) and s["c3"].zipf_s == 1.2
    assert s["c4"].ops == ((1, 16384), (0, 256)) and s["c4"].layers == 8
    assert s["c5"].shape == synth.Shape(256, 8, 6144, 2048, "fp8")


def test_routing_valid_and_deterministic():
    for name in ("c1", "c2", "c3", "c5"):
        spec = synth.SPECS[name]
        for i, (cls, T) in enumerate(spec.ops):
            T = min(T, 512)
            ids, w = synth.make_routing(spec, T, 0, i)
            ids2, w2 = synth.make_routing(spec, T, 0, i)
            assert np.array_equal(ids, ids2) and np.array_equal(w, w2)
            assert ids.dtype == np.int32 and w.dtype == np.float32
            assert ids.min() >= 0 and ids.max() < spec.shape.E
            assert all(len(set(r)) == spec.shape.k for r in ids)          # distinct experts
            assert np.allclose(w.sum(1), 1.0, atol=1e-5) and np.all(np.diff(w, axis=1) <= 0)


def test_zipf_is_skewed_and_layers_shift_load():
    spec = synth.SPECS["c4"]
    hist = []
    for layer in range(3):
        ids, _ = synth.make_routing(spec, 4096, layer, 0)
        c = np.bincount(ids.reshape(-1), minlength=256)
        assert c.max() > 8 * np.median(c)
        hist.append(np.argsort(-c)[:8])
        assert 0.6 <= synth.layer_zipf_s(spec, layer) <= 1.6
    assert not np.array_equal(hist[0], hist[1])                            # fresh expert order


def test_tensors_deterministic_and_fp8_blocks():
    spec = synth.scaled(synth.SPECS["c5"], shape=synth.Shape(2, 2, 256, 128, "fp8"),
                        ops=((synth.PREFILL, 4),))
    a, b = synth.make_weights(spec, threads=1), synth.make_weights(spec, threads=2)
    assert torch.equal(a.w_gate_up, b.w_gate_up) and torch.equal(a.s_down, b.s_down)
    assert a.w_gate_up.dtype == torch.uint8 and a.s_gate_up.shape == (2, 2, 2)
    v = a.w_gate_up.view(torch.float8_e4m3fn).float().view(2, 2, 128, 2, 128)
    assert torch.all(v.abs().amax(dim=(2, 4)) == 448.0)                    # amax maps to 448
    x, xs = synth.make_x(spec, 4, 0, 0)
    assert x.shape == (4, 256) and xs.shape == (4, 2)
    c1 = synth.make_weights(synth.SPECS["c1"], threads=1)
    assert c1.w_gate_up.dtype == torch.bfloat16 and c1.w_gate_up.shape == (8, 1024, 256)
    assert abs(c1.w_gate_up.float().std().item() - 0.02) < 1e-3


def test_route_active_pool_uses_exactly_the_pool():
    rng = np.random.default_rng(3)
    ids, w = synth.route_active_pool(rng, 64, 4, 32, 8)
    assert ids.shape == (64, 4) and len(np.unique(ids)) == 8
    assert all(len(set(r)) == 4 for r in ids.tolist())
    assert np.allclose(w.sum(axis=1), 1.0, atol=1e-6)
    with pytest.raises(ValueError):
        synth.route_active_pool(rng, 4, 4, 32, 2)


def test_latency_model_fit_recovers_an_affine_law():
    from paper_2607_18002_b200.latency_model import fit_affine
    x = np.array([8, 16, 32, 64, 128, 256], dtype=np.float64)
    a, b, r2 = fit_affine(x, 40.0 + 4.5 * x)
    assert abs(a - 40.0) < 1e-9 and abs(b - 4.5) < 1e-9 and r2 > 1 - 1e-12
    rng = np.random.default_rng(0)
    a, b, r2 = fit_affine(x, 40.0 + 4.5 * x + rng.normal(0, 1.0, x.shape))
    assert abs(b - 4.5) < 0.1 and r2 > 0.99
