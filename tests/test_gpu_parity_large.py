"""Parity at the larger configurations on subsets the oracle can afford (sequences are independent, so a batch row
checked alone against a batch-1 oracle is a full check of that row)."""
import copy

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


def _weights_gpu(shape, seed, torch):
    """bf16 weights drawn on the GPU (N(0, 0.02^2)); returned as torch tensors and as float32 numpy for the oracle."""
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    w = {k: (torch.randn((shape.d_model, shape.d_model), generator=gen, device="cuda") * 0.02).to(torch.bfloat16)
         for k in ("w_q", "w_k", "w_v", "w_o")}
    w["rms_gain"] = torch.ones(shape.d_model, device="cuda")
    wn = {k: v.float().cpu().numpy() for k, v in w.items()}
    return w, wn


def test_config3_dare_o_batched_clustered_steps(dare):
    """Config 3: batch 8, seq 1024, mode O, 113 clustered + 20 scattered positions changed per sequence and step, 64
    consecutive denoising steps on one handle (the active block moves every four steps, sixteen blocks).
    All 8 sequences run on the GPU; sequences 0 and 5 are checked against batch-1 oracles at every step (layer output,
    index list, staleness counters; the K and O caches every eighth step and at the end); the index sets of all
    sequences are checked against the plan at every step."""
    import torch
    shape = wl.LLADA_DARE_O
    w_t, w_np = _weights_gpu(shape, 33, torch)
    hs = wl.HiddenStream(shape)
    g = dare.Layer(shape, w_t)
    one = wl.scaled(shape, batch=1)
    checked = (0, 5)
    oracles = {b: parity.oracle_layer(one, w_np) for b in checked}
    x = hs.first()
    y = g.step(parity.to_device(x, shape), 2, 0.1)
    yo = {b: oracles[b].step(x[b:b + 1], 2, 0.1) for b in checked}
    for b in checked:
        parity.assert_close(f"y step0 seq{b}", y[b:b + 1].float().cpu().numpy(), yo[b], parity.TOL_BF16, rel_rms=parity.TOL_BF16)
    n_steps = 64
    for step in range(1, n_steps + 1):
        ch = wl.clustered_positions(hs.rng, shape, step - 1, 113, 20)
        x = hs.advance(ch)
        y = g.step(parity.to_device(x, shape), 2, 0.1)
        sel = g.last_selection(shape.batch, shape.seq)
        np.testing.assert_array_equal(sel["idx"], np.nonzero(ch.reshape(-1))[0])
        assert sel["count"] == 133 * shape.batch
        np.testing.assert_array_equal(np.diff(sel["batch_off"]), np.full(shape.batch, 133))
        with_caches = step % 8 == 0 or step == n_steps
        caches = g.read_caches(shape.batch, shape.seq) if with_caches else None
        yh = y.float().cpu().numpy()
        for b in checked:
            o = oracles[b]
            yo_b = o.step(x[b:b + 1], 2, 0.1)
            parity.check_margin(o.last_scores, 0.1)
            np.testing.assert_array_equal(sel["idx"][sel["batch_off"][b]:sel["batch_off"][b + 1]] - b * shape.seq, o.last_idx)
            parity.assert_close(f"y step{step} seq{b}", yh[b:b + 1], yo_b, parity.TOL_BF16, rel_rms=parity.TOL_BF16)
            np.testing.assert_array_equal(sel["delta"][b], o.delta[0])
            if with_caches:
                parity.assert_close(f"o_cache step{step} seq{b}", caches["o"][b:b + 1], o.o_cache, parity.TOL_BF16, max_factor=2.0)
                parity.assert_close(f"k_cache step{step} seq{b}", caches["k"][b:b + 1], o.k_cache, parity.TOL_BF16, max_factor=2.0)
    # after 64 steps some rows have been reused for dozens of steps in a row, others were refreshed in the last one
    assert sel["delta"].max() >= 32 and (sel["delta"] == 0).sum() == 133 * shape.batch
    assert g.status() == 0
    g.close()


@pytest.fixture(scope="module")
def config5(dare):
    """Config 5 (batch 4, seq 4096): weights, the first hidden states, a GPU layer, and a batch-1 oracle of sequence 2
    after its first step (dense whatever the mode, so one oracle state serves every case)."""
    import torch
    shape = wl.LLADA_LONG
    w_t, w_np = _weights_gpu(shape, 55, torch)
    hs = wl.HiddenStream(shape)
    x0 = hs.first()
    g = dare.Layer(shape, w_t)
    b = 2
    o0 = parity.oracle_layer(wl.scaled(shape, batch=1), w_np)
    y0 = o0.step(x0[b:b + 1], 3, 0.1)
    yield shape, g, hs, x0, parity.to_device(x0, shape), b, o0, y0
    g.close()


def _changed(hs, shape, frac, pattern):
    n = int(round(frac * shape.seq))
    if n == 0:
        return np.zeros((shape.batch, shape.seq), bool)
    return wl.uniform_positions(hs.rng, shape, n) if pattern == "uniform" else wl.clustered_positions(hs.rng, shape, 9, n, 0)


@pytest.mark.parametrize("frac,pattern,mode", [(0.0, "uniform", 3), (0.0, "clustered", 2), (0.15, "uniform", 3),
                                               (0.15, "clustered", 2), (0.5, "uniform", 2), (0.5, "clustered", 1),
                                               (1.0, "uniform", 1), (1.0, "clustered", 3)])
def test_config5_long_context_one_sequence(dare, config5, frac, pattern, mode):
    """Config 5: changed fractions 0, 15, 50 and 100 % in both patterns, every reuse mode; all four sequences run on the
    GPU, sequence 2 is checked against the batch-1 oracle (layer output, K, V and O caches, index list, staleness),
    the index sets of all sequences against the plan."""
    shape, g, hs0, x0, x0_dev, b, o0, y0 = config5
    hs = copy.deepcopy(hs0)
    g.reset()
    yg0 = g.step(x0_dev, mode, 0.1)
    parity.assert_close("y step0", yg0[b:b + 1].float().cpu().numpy(), y0, parity.TOL_BF16, rel_rms=parity.TOL_BF16)
    ch = _changed(hs, shape, frac, pattern)
    x1 = hs.advance(ch)
    y1 = g.step(parity.to_device(x1, shape), mode, 0.1)
    sel = g.last_selection(shape.batch, shape.seq)
    np.testing.assert_array_equal(sel["idx"], np.nonzero(ch.reshape(-1))[0])
    o = copy.deepcopy(o0)
    yo = o.step(x1[b:b + 1], mode, 0.1)
    parity.check_margin(o.last_scores, 0.1)
    np.testing.assert_array_equal(sel["idx"][sel["batch_off"][b]:sel["batch_off"][b + 1]] - b * shape.seq, o.last_idx)
    np.testing.assert_array_equal(sel["delta"][b], o.delta[0])
    parity.assert_close("y step1", y1[b:b + 1].float().cpu().numpy(), yo, parity.TOL_BF16, rel_rms=parity.TOL_BF16)
    caches = g.read_caches(shape.batch, shape.seq)
    parity.assert_close("k_cache", caches["k"][b:b + 1], o.k_cache, parity.TOL_BF16, max_factor=2.0)
    parity.assert_close("v_cache", caches["v"][b:b + 1], o.v_cache, parity.TOL_BF16, max_factor=2.0)
    parity.assert_close("o_cache", caches["o"][b:b + 1], o.o_cache, parity.TOL_BF16, max_factor=2.0)
    assert g.status() == 0


@pytest.mark.parametrize("pattern", ["uniform", "clustered"])
def test_config5_index_sets_over_the_whole_sweep(dare, config5, pattern):
    """The 21 points of the crossover sweep (0 to 100 % changed in steps of 5 %): the GPU's index list of every
    sequence against the plan, and that of sequence 2 against the oracle's scores (lines 1-3 of Alg. 1 and Eq. 2 only,
    which is all an index set needs), with the margin checked on those scores."""
    from oracle import dare_oracle as orc
    shape, g, hs0, x0, x0_dev, b, o0, y0 = config5
    for i in range(21):
        frac = 0.05 * i
        hs = copy.deepcopy(hs0)
        hs.rng = np.random.default_rng(1000 * i + (0 if pattern == "uniform" else 500))
        g.reset()
        g.step(x0_dev, 3, 0.1)
        ch = _changed(hs, shape, frac, pattern)
        x1 = hs.advance(ch)
        g.step(parity.to_device(x1, shape), 3, 0.1)
        sel = g.last_selection(shape.batch, shape.seq)
        assert sel["count"] == int(ch.sum()) == shape.batch * int(round(frac * shape.seq))
        np.testing.assert_array_equal(sel["idx"], np.nonzero(ch.reshape(-1))[0])
        s = orc.scores_only(o0, x1[b:b + 1])
        parity.check_margin(s, 0.1)
        want = np.nonzero(orc.refresh_mask(s, 0.1))[0]
        np.testing.assert_array_equal(sel["idx"][sel["batch_off"][b]:sel["batch_off"][b + 1]] - b * shape.seq, want)
        np.testing.assert_allclose(sel["scores"][b * shape.seq:(b + 1) * shape.seq], s, rtol=0,
                                   atol=parity.SCORE_ATOL[wl.DTYPE_BF16])
    assert g.status() == 0


@pytest.mark.parametrize("pattern", ["uniform", "clustered"])
def test_listed_and_dense_forms_on_both_sides_of_their_gates(dare, pattern):
    """A step of many row tiles issues its K/V projection, its attention and its output projection in two forms, listed
    (over the refresh set) and dense (over every row, results kept for the refreshed rows only), and the size of the
    refresh set decides on the device which runs: from 75 % of the tokens on for the K/V projection, from 80 % for the
    other two.  Width 2048, 2 x 2560 tokens (40 row tiles: every projection in the persistent kernel); consecutive steps
    at 30, 78, 90, 100, 77 and 85 % changed in rotating modes, checked against the oracle in full: the forms must give
    the same caches and outputs, and reused rows must stay untouched, whichever side of a gate a step falls on."""
    shape = wl.scaled(wl.LLADA_LAYER, d_model=2048, n_heads=16, batch=2, seq=2560, prompt=1280)
    w = wl.make_weights(shape, 71)
    hs = wl.HiddenStream(shape, 71)
    g = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    o = parity.oracle_layer(shape, w)
    parity.compare_step(g, o, hs.first(), 3, 0.1, shape, first=True)
    for i, frac in enumerate((0.30, 0.78, 0.90, 1.00, 0.77, 0.85)):
        n = int(round(frac * shape.seq))
        ch = (wl.uniform_positions(hs.rng, shape, n) if pattern == "uniform"
              else wl.clustered_positions(hs.rng, shape, 4 * i, n, 0))
        before = g.read_caches(shape.batch, shape.seq)
        mode = (3, 3, 3, 3, 1, 2)[i]
        parity.compare_step(g, o, hs.advance(ch), mode, 0.1, shape)
        after = g.read_caches(shape.batch, shape.seq)
        keep = ~ch
        if mode & 1:
            assert np.array_equal(after["k"][keep], before["k"][keep]) and np.array_equal(after["v"][keep], before["v"][keep])
        if mode & 2:
            assert np.array_equal(after["o"][keep], before["o"][keep])
        assert g.last_selection(shape.batch, shape.seq)["count"] == n * shape.batch
    assert g.status() == 0
    g.close()


def test_long_context_attention_repeats_bit_identically(dare):
    """Batch 4 x 4096, two steps (dense, then K/V reuse at 50 % clustered) on three fresh handles: the caches must be
    bit-identical from run to run.  The softmax warps of the two-tile attention kernel run up to two P V products
    ahead of the tensor core there; a wait that mistook one phase of a barrier for another showed up as outputs that
    varied between runs."""
    import torch
    shape = wl.LLADA_LONG
    w_t, _ = _weights_gpu(shape, 55, torch)

    def run():
        hs = wl.HiddenStream(shape)
        g = dare.Layer(shape, w_t)
        g.step(parity.to_device(hs.first(), shape), 1, 0.1)
        c0 = g.read_caches(shape.batch, shape.seq)
        ch = wl.clustered_positions(hs.rng, shape, 9, shape.seq // 2, 0)
        g.step(parity.to_device(hs.advance(ch), shape), 1, 0.1)
        c1 = g.read_caches(shape.batch, shape.seq)
        assert g.status() == 0
        g.close()
        return c0, c1

    a0, a1 = run()
    for _ in range(2):
        b0, b1 = run()
        for name in ("k", "v", "o"):
            np.testing.assert_array_equal(a0[name], b0[name])
            np.testing.assert_array_equal(a1[name], b1[name])
