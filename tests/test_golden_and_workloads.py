"""The stored config-1 oracle values still come out of the oracle, and the generators keep their contract."""
import importlib.util
import json
import os

import numpy as np

from paper_2605_08134_b200 import workloads as wl

HERE = os.path.dirname(os.path.abspath(__file__))


def _load_maker():
    spec = importlib.util.spec_from_file_location("make_config1_golden", os.path.join(HERE, "golden", "make_config1_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_config1_golden_reproduces():
    with open(os.path.join(HERE, "golden", "config1_oracle.json")) as f:
        stored = json.load(f)
    fresh = _load_maker().build()
    assert fresh["planned"] == stored["planned"]
    for name in ("kv", "o", "both"):
        a, b = fresh["modes"][name], stored["modes"][name]
        assert a["idx"] == b["idx"] == stored["planned"]
        # margins of config 1: every score at least 1e-3 away from tau = 0.1
        assert b["score_min_selected"] - 0.1 >= 1e-3 and 0.1 - b["score_max_reused"] >= 1e-3
        for key in ("y0_samples", "y1_samples"):
            np.testing.assert_allclose(a[key], b[key], rtol=1e-9, atol=1e-12)
        for key in ("y1_rms", "y1_sum", "k_cache_sum", "o_cache_sum"):
            np.testing.assert_allclose(a[key], b[key], rtol=1e-9, atol=1e-9)


def test_bf16_rounding_is_nearest_even():
    # 1 + 2^-8 is halfway between bf16 neighbours 1 and 1 + 2^-7: ties go to the even mantissa (1.0)
    a = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0, 3.0e38], np.float32)
    r = wl.bf16_round(a)
    np.testing.assert_array_equal(r[:4], np.array([1.0, 1.0, 1.0 + 2.0 ** -7, 1.0 + 2.0 ** -6], np.float32))
    assert r[4] == -2.5 and r[5] == 0.0 and np.isfinite(r[6])
    import torch
    x = np.random.default_rng(0).standard_normal(4096).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(wl.bf16_round(x), ref)
    np.testing.assert_array_equal(wl.bf16_bits_to_f32(wl.bf16_bits(x)), ref)


def test_streams_are_seeded_and_structured():
    shape = wl.scaled(wl.LLADA_DARE_O, d_model=64, n_heads=2, head_dim=32, batch=2, seq=256, prompt=128)
    a, b = wl.HiddenStream(shape), wl.HiddenStream(shape)
    np.testing.assert_array_equal(a.first(), b.first())
    m = wl.clustered_positions(a.rng, shape, step=5, clustered_per_seq=28, scattered_per_seq=5)
    assert m.shape == (2, 256) and (m.sum(axis=1) == 33).all()
    start = shape.prompt + (5 // 4) * shape.block
    assert m[:, start:start + 28].all()
    x1 = a.advance(m)
    x0 = wl.round_to(b.master, shape.dtype)
    moved = np.abs(x1 - x0).max(axis=-1)
    assert (moved[m] > 0.5).all() and (moved[~m] < 0.1).all()
    # bf16 storage: every value is representable
    np.testing.assert_array_equal(wl.bf16_round(x1), x1)
    # wrap-around of the clustered run stays inside the generation region
    m2 = wl.clustered_positions(a.rng, shape, step=15, clustered_per_seq=60, scattered_per_seq=0)
    assert not m2[:, :shape.prompt].any() and (m2.sum(axis=1) == 60).all()


def test_weights_follow_the_recipe():
    w = wl.make_weights(wl.TINY_F32)
    for k in ("w_q", "w_k", "w_v", "w_o"):
        assert w[k].shape == (256, 256) and abs(w[k].std() - 0.02) < 1e-3 and abs(w[k].mean()) < 1e-3
    assert (w["rms_gain"] == 1).all()
    w2 = wl.make_weights(wl.scaled(wl.LLADA_LAYER, d_model=128, n_heads=1))
    np.testing.assert_array_equal(wl.bf16_round(w2["w_q"]), w2["w_q"])
