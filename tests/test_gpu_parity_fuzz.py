"""Seeded random geometries through the tensor-core path against the fp64 oracle: odd sequence lengths and windows,
every mode, refresh sets from empty to full.  The sizes walk across the launch rules of the kernels (split-K or not,
128- or 256-wide gathered tiles, one or two query tiles per attention CTA, key split, gathered output projection,
short or long selection, two-CTA MMAs with an even or odd number of row tiles)."""
import numpy as np
import pytest

from paper_2605_08134_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dare():
    from paper_2605_08134_b200 import build
    build.build()
    from paper_2605_08134_b200 import dare as d
    return d


CASES = [
    # d_model, batch, seq, prompt
    (256, 1, 57, 20),
    (256, 3, 129, 1),
    (512, 2, 700, 188),
    (256, 1, 2300, 252),        # few (head, sequence) pairs, many key blocks: key split
    (512, 5, 1031, 7),          # > 8 row tiles: gathered output projection, 256-wide gathered tiles
    (1024, 8, 1153, 129),       # two query tiles per attention CTA, dense and row-sparse
    (1024, 2, 384, 128),
    (256, 6, 513, 100),
    (256, 3, 100, 10),          # three row tiles: MMA pairs with a padding tile, split reduction
    (512, 1, 384, 64),
    (512, 1, 100, 10),
    (1024, 2, 256, 64),
    (512, 16, 1153, 100),       # 160 row tiles at a short reduction: every projection in the persistent kernel
    (1024, 1, 250, 60),         # two row tiles: narrow MMA-pair tiles (one sequence, ragged)
    (512, 2, 128, 32),          # ... one row tile per sequence
    (4096, 1, 250, 100),        # the full layer width at two, two and three row tiles: narrow pairs, padding tile
    (4096, 2, 128, 16),
    (4096, 3, 120, 20),
]


@pytest.mark.parametrize("case", range(len(CASES)))
def test_random_steps(dare, case):
    d_model, batch, seq, prompt = CASES[case]
    rng = np.random.default_rng(1000 + case)
    shape = wl.scaled(wl.LLADA_LAYER, d_model=d_model, n_heads=d_model // 128, batch=batch, seq=seq, prompt=prompt)
    w = wl.make_weights(shape, 300 + case)
    hs = wl.HiddenStream(shape, 300 + case)
    g = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    o = parity.oracle_layer(shape, w)
    parity.compare_step(g, o, hs.first(), int(rng.integers(0, 4)), 0.1, shape, first=True)
    for step in range(4):
        mode = int(rng.integers(0, 4))
        frac = float(rng.choice([0.0, 0.03, 0.13, 0.4, 1.0]))
        n = min(seq, int(round(frac * seq)))
        ch = wl.uniform_positions(hs.rng, shape, n) if n > 0 else np.zeros((batch, seq), bool)
        x = hs.advance(ch)
        if rng.random() < 0.5:
            parity.compare_step(g, o, x, mode, 0.1, shape)
        else:
            parity.compare_step(g, o, np.ascontiguousarray(x[:, prompt:]), mode, 0.1, shape, pos_begin=prompt)
    g.close()


BIG = [(512, 5, 3892, 1075), (1024, 5, 3196, 3030), (4096, 2, 2159, 564)]


@pytest.mark.parametrize("case", range(len(BIG)))
def test_large_geometries_repeat_bit_identically(dare, case):
    """Shapes of several thousand rows (persistent projections in their one- and two-CTA forms, listed launches, two query
    tiles per attention CTA): two fresh handles through the same four steps give bit-identical outputs and caches."""
    import torch
    d_model, batch, seq, prompt = BIG[case]
    shape = wl.scaled(wl.LLADA_LAYER, d_model=d_model, n_heads=d_model // 128, batch=batch, seq=seq, prompt=prompt)
    w = wl.make_weights(shape, 800 + case)
    hs = wl.HiddenStream(shape, 800 + case)
    rng = np.random.default_rng(6000 + case)
    steps = [(hs.first(), int(rng.integers(0, 4)), 0)]
    for _ in range(3):
        mode = int(rng.integers(0, 4))
        n = max(1, int(round(float(rng.choice([0.03, 0.13, 0.4, 1.0])) * seq)))
        x = hs.advance(wl.uniform_positions(hs.rng, shape, n))
        if rng.random() < 0.4:
            steps.append((np.ascontiguousarray(x[:, prompt:]), mode, prompt))
        else:
            steps.append((x, mode, 0))
    outs = []
    for _ in range(2):
        g = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
        ys = [g.step(parity.to_device(x, shape), mode, 0.1, pos_begin=pb).clone() for x, mode, pb in steps]
        torch.cuda.synchronize()
        caches = g.read_caches(batch, seq)
        assert g.status() == 0
        g.close()
        outs.append((ys, caches))
    for a, b in zip(outs[0][0], outs[1][0]):
        assert torch.equal(a, b)
    for name in ("k", "v", "o"):
        np.testing.assert_array_equal(outs[0][1][name], outs[1][1][name])
