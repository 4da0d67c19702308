"""GPU parity of the tensor-core kernel path (tcgen05 / TMEM / TMA) against the fp64 oracle."""
import copy

import numpy as np
import pytest

from paper_2605_08134_b200 import workloads as wl
from tests import parity, rounding

pytestmark = pytest.mark.gpu

MODES = {"kv": 1, "o": 2, "both": 3, "dense": 0}


@pytest.fixture(scope="module")
def dare():
    from paper_2605_08134_b200 import build
    build.build()
    from paper_2605_08134_b200 import dare as d
    return d


@pytest.mark.parametrize("mode", list(MODES))
def test_small_llada_shaped_layer_ragged(dare, mode):
    """4 heads x 128, batch 2, seq 320 (2.5 row tiles per sequence), three steps."""
    shape = wl.scaled(wl.LLADA_LAYER, d_model=512, n_heads=4, batch=2, seq=320, prompt=160)
    w = wl.make_weights(shape, 21)
    hs = wl.HiddenStream(shape, 21)
    g = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    o = parity.oracle_layer(shape, w)
    parity.compare_step(g, o, hs.first(), MODES[mode], 0.1, shape, first=True)
    for t in range(2):
        ch = wl.uniform_positions(hs.rng, shape, (41, 150)[t])
        parity.compare_step(g, o, hs.advance(ch), MODES[mode], 0.1, shape)
        if mode != "dense":
            np.testing.assert_array_equal(g.last_selection(2, 320)["idx"], np.nonzero(ch.reshape(-1))[0])
    g.close()


def test_tensor_path_agrees_with_cuda_core_path(dare):
    shape = wl.scaled(wl.LLADA_LAYER, d_model=256, n_heads=2, batch=1, seq=200, prompt=100)
    w, x0, x1, ch = wl.two_step_case(shape, 30, seed=8)
    a = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    b = dare.Layer(shape, w, kernel_path=dare.PATH_SIMT)
    for x in (x0, x1):
        ya = a.step(parity.to_device(x, shape), 3, 0.1)
        yb = b.step(parity.to_device(x, shape), 3, 0.1)
        parity.assert_close("tensor vs cuda-core", ya.float().cpu().numpy(), yb.float().cpu().numpy(), 2e-2)
    np.testing.assert_array_equal(a.last_selection(1, 200)["idx"], b.last_selection(1, 200)["idx"])
    a.close(); b.close()


def test_window_steps_tensor_path(dare):
    shape = wl.scaled(wl.LLADA_LAYER, d_model=256, n_heads=2, batch=2, seq=288, prompt=128)
    w = wl.make_weights(shape, 6)
    hs = wl.HiddenStream(shape, 6)
    g = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    o = parity.oracle_layer(shape, w)
    parity.compare_step(g, o, hs.first(), 3, 0.1, shape, first=True)
    p = shape.prompt
    for t in range(3):
        ch = wl.uniform_positions(hs.rng, shape, 30)
        x = hs.advance(ch)
        parity.compare_step(g, o, np.ascontiguousarray(x[:, p:]), (3, 1, 2)[t], 0.1, shape, pos_begin=p)
    g.close()


@pytest.fixture(scope="module")
def config2():
    shape = wl.LLADA_LAYER
    w = wl.make_weights(shape)
    hs = wl.HiddenStream(shape)
    x0 = hs.first()
    o = parity.oracle_layer(shape, w)
    y0 = o.step(x0, 0, 0.1)
    return shape, w, hs, x0, o, y0


@pytest.mark.parametrize("n_changed", [26, 67, 154, 256, 330, 512])
def test_config2_llada_layer_full_size(dare, config2, n_changed):
    """Config 2: d=4096, 32 heads x 128, seq 512, bf16; changed fraction 5/13/30/50/100 %, all three reuse modes
    (and 330 rows: three row tiles, of which the gathered projection's clusters take two in one pass and share the third)."""
    shape, w, hs0, x0, o0, y0 = config2
    hs = copy.deepcopy(hs0)
    ch = wl.uniform_positions(hs.rng, shape, n_changed)
    x1 = hs.advance(ch)
    g = dare.Layer(shape, w)
    assert g.cfg.kernel_path == dare.PATH_AUTO
    for mode in ("both", "kv", "o"):
        g.reset()
        yg = g.step(parity.to_device(x0, shape), MODES[mode], 0.1)
        parity.assert_close("y step0", yg.float().cpu().numpy(), y0, parity.TOL_BF16)
        o = copy.deepcopy(o0)
        parity.compare_step(g, o, x1, MODES[mode], 0.1, shape)
        np.testing.assert_array_equal(g.last_selection(1, 512)["idx"], np.nonzero(ch.reshape(-1))[0])
    g.close()


def test_row_sparse_attention_with_key_split(dare):
    """Batch 1, 2 heads, 2048 keys, few refreshed rows: the row-sparse attention launch splits the keys over a 4-CTA
    cluster and merges the partial softmax results over distributed shared memory."""
    shape = wl.scaled(wl.LLADA_LAYER, d_model=256, n_heads=2, batch=1, seq=2048, prompt=1024)
    w = wl.make_weights(shape, 13)
    hs = wl.HiddenStream(shape, 13)
    g = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    o = parity.oracle_layer(shape, w)
    parity.compare_step(g, o, hs.first(), 3, 0.1, shape, first=True)
    for n in (37, 150):
        ch = wl.uniform_positions(hs.rng, shape, n)
        parity.compare_step(g, o, hs.advance(ch), 3, 0.1, shape)
    # a ragged key extent as well: window steps keep kv_len = 2048, so use a second layer with 1990 keys
    shape2 = wl.scaled(shape, seq=1990, prompt=990)
    hs2 = wl.HiddenStream(shape2, 14)
    g2 = dare.Layer(shape2, w, kernel_path=dare.PATH_TENSOR)
    o2 = parity.oracle_layer(shape2, w)
    parity.compare_step(g2, o2, hs2.first(), 2, 0.1, shape2, first=True)
    parity.compare_step(g2, o2, hs2.advance(wl.uniform_positions(hs2.rng, shape2, 70)), 2, 0.1, shape2)
    g.close(); g2.close()


def test_single_key_block(dare):
    """kv_len below one key block: one of the attention kernel's two key-block streams has nothing to do."""
    shape = wl.scaled(wl.LLADA_LAYER, d_model=256, n_heads=2, batch=2, seq=96, prompt=32)
    w = wl.make_weights(shape, 12)
    hs = wl.HiddenStream(shape, 12)
    g = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    o = parity.oracle_layer(shape, w)
    parity.compare_step(g, o, hs.first(), 3, 0.1, shape, first=True)
    for mode in (3, 2, 0):
        parity.compare_step(g, o, hs.advance(wl.uniform_positions(hs.rng, shape, 17)), mode, 0.1, shape)
    g.close()


def test_peaked_softmax_rescales_the_accumulator(dare):
    """Sharp attention (large query/key projections): the running row maximum of a key-block stream jumps by more
    than the kernel's lazy-rescaling step (2^8), so the in-place rescale of the tensor-memory accumulator runs.
    The jump is checked on the oracle's own scores.  With logits this large the bf16 rounding of the stored Q and K
    decides the distance to the plain fp64 oracle: a logit of size |l| moves by about |l| * 2^-8 / sqrt(3 * 128) * sqrt(2),
    a few 1e-2 here, and a softmax weight by that relative amount, whatever the kernel does with the rounded operands.
    The tensor path is therefore held, at the ordinary bf16 tolerance, to the oracle's arithmetic evaluated in fp64 on
    the tensors as the kernels store them (x_norm, rotated Q, K, V and attention output rounded to bf16:
    tests/rounding.py), and to the CUDA-core path, which shares those operands; the index set is held to the plain
    oracle."""
    from oracle import dare_oracle as orc
    shape = wl.scaled(wl.LLADA_LAYER, d_model=256, n_heads=2, batch=1, seq=1280, prompt=640)
    w = wl.make_weights(shape, 44)
    for k in ("w_q", "w_k"):
        w[k] = wl.round_to(w[k] * np.float32(6.0), shape.dtype)
    hs = wl.HiddenStream(shape, 44)
    x0 = hs.first()
    ch = wl.uniform_positions(hs.rng, shape, 150)
    x1 = hs.advance(ch)
    # the oracle's logits of step 0: does some row's maximum over the blocks of one stream grow by > 8 / log2(e)?
    xn = orc.rmsnorm(x0[0], w["rms_gain"], shape.rms_eps)
    pos = np.arange(shape.seq)
    q = orc.rope(orc.linear(xn, w["w_q"]), pos, shape.n_heads, shape.head_dim, shape.rope_theta)
    k = orc.rope(orc.linear(xn, w["w_k"]), pos, shape.n_heads, shape.head_dim, shape.rope_theta)
    jumps = 0
    for h in range(shape.n_heads):
        sl = slice(h * 128, (h + 1) * 128)
        logit = q[:, sl] @ k[:, sl].T / np.sqrt(128.0)
        blockmax = logit.reshape(shape.seq, shape.seq // 128, 128).max(axis=2)      # [row, block]
        for st in range(2):
            bm = blockmax[:, st::2]
            run = np.maximum.accumulate(bm, axis=1)
            jumps += int(((run[:, 1:] - run[:, :-1]) > 8.0 / np.log2(np.e)).sum())
    assert jumps > 50, jumps
    a = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    b = dare.Layer(shape, w, kernel_path=dare.PATH_SIMT)
    o = parity.oracle_layer(shape, w)
    r = rounding.rounded_layer(shape, w)
    for x, mode in ((x0, 0), (x1, 3)):
        ya = a.step(parity.to_device(x, shape), mode, 0.1)
        yb = b.step(parity.to_device(x, shape), mode, 0.1)
        o.step(x, mode, 0.1)
        yr = r.step(x, mode, 0.1)
        parity.assert_close("tensor vs cuda-core", ya.float().cpu().numpy(), yb.float().cpu().numpy(), 2e-2)
        parity.assert_close("tensor vs oracle on stored operands", ya.float().cpu().numpy(), yr, parity.TOL_BF16,
                            rel_rms=parity.TOL_BF16)
        parity.assert_close("o_cache vs oracle on stored operands", a.read_caches(1, shape.seq)["o"], r.o_cache[:1],
                            parity.TOL_BF16)
        np.testing.assert_array_equal(r.last_idx, o.last_idx)
    np.testing.assert_array_equal(a.last_selection(1, shape.seq)["idx"], o.last_idx)
    np.testing.assert_array_equal(a.last_selection(1, shape.seq)["idx"], b.last_selection(1, shape.seq)["idx"])
    a.close(); b.close()


def test_gathered_output_projection_windows_and_state(dare):
    """Many tokens per step (more than eight row tiles): on steps that reuse attention outputs the output projection
    runs over the refresh set only and the other rows come from the cache of projected rows.  Checked against the
    oracle over full-extent and window steps in every mode, and across an export/import of the layer state (which
    does not carry that cache: the next step projects every row again)."""
    import torch
    shape = wl.scaled(wl.LLADA_LAYER, d_model=256, n_heads=2, batch=2, seq=1280, prompt=256)
    w = wl.make_weights(shape, 31)
    hs = wl.HiddenStream(shape, 31)
    g = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    o = parity.oracle_layer(shape, w)
    parity.compare_step(g, o, hs.first(), 3, 0.1, shape, first=True)
    parity.compare_step(g, o, hs.advance(wl.uniform_positions(hs.rng, shape, 200)), 3, 0.1, shape)
    p = shape.prompt
    for mode in (2, 1, 3):            # window of 1024 positions x 2 sequences = 16 row tiles
        x = hs.advance(wl.uniform_positions(hs.rng, shape, 120))
        parity.compare_step(g, o, np.ascontiguousarray(x[:, p:]), mode, 0.1, shape, pos_begin=p)
    # nothing refreshed (every row copied from the cache of projected rows), then everything refreshed
    for tau in (float("inf"), -1.0):
        x = hs.advance(wl.uniform_positions(hs.rng, shape, 60))
        parity.compare_step(g, o, np.ascontiguousarray(x[:, p:]), 3, tau, shape, pos_begin=p)
    # state to a second handle: same results from there on
    n = dare.dare_layer_state_bytes(g.handle)
    blob = torch.empty(n, dtype=torch.uint8).pin_memory()
    assert dare.dare_layer_export_state(g.handle, blob.data_ptr(), n) == 0
    g2 = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    assert dare.dare_layer_import_state(g2.handle, blob.data_ptr(), n) == 0
    for mode in (2, 3):
        x = hs.advance(wl.uniform_positions(hs.rng, shape, 90))
        xw = np.ascontiguousarray(x[:, p:])
        y2 = g2.step(parity.to_device(xw, shape), mode, 0.1, pos_begin=p)
        _, yo = parity.compare_step(g, o, xw, mode, 0.1, shape, pos_begin=p)
        np.testing.assert_array_equal(g2.last_selection(2, shape.seq - p)["idx"], o.last_idx)
        parity.assert_close("imported handle y", y2.float().cpu().numpy(), yo, 2e-2)
    g.close(); g2.close()


def test_two_tile_attention_ragged(dare):
    """Sizes that send dense and row-sparse attention to the kernel with two query tiles per CTA (many rows per
    sequence and enough (head, sequence) pairs to fill the GPU), with everything ragged: 1100 keys (8 blocks + 76),
    windows whose last 256-row tile holds 76 rows (its second tile empty), refresh sets that end inside a tile."""
    shape = wl.scaled(wl.LLADA_LAYER, d_model=1024, n_heads=8, batch=8, seq=1100, prompt=76)
    w = wl.make_weights(shape, 52)
    hs = wl.HiddenStream(shape, 52)
    g = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    o = parity.oracle_layer(shape, w)
    parity.compare_step(g, o, hs.first(), 3, 0.1, shape, first=True)
    parity.compare_step(g, o, hs.advance(wl.uniform_positions(hs.rng, shape, 300)), 3, 0.1, shape)
    p = shape.prompt
    for mode, n in ((2, 150), (0, 10)):   # window of 1024 positions: row-sparse, then dense
        x = hs.advance(wl.uniform_positions(hs.rng, shape, n))
        parity.compare_step(g, o, np.ascontiguousarray(x[:, p:]), mode, 0.1, shape, pos_begin=p)
    g.close()


@pytest.mark.parametrize("geom", ["llada_layer", "many_tokens"])
def test_tensor_path_is_deterministic(dare, geom):
    """Two handles, same weights, same steps: bit-identical outputs and caches (fixed reduction orders in the split-K
    exchange, the stream merge and the key split; no result depends on scheduling)."""
    import torch
    if geom == "llada_layer":
        shape = wl.LLADA_LAYER
        changed, modes = 67, (3, 3, 2, 1, 0)
    else:
        shape = wl.scaled(wl.LLADA_LAYER, d_model=1024, n_heads=8, batch=8, seq=1280, prompt=256)
        changed, modes = 200, (3, 2, 3, 1, 0)
    w = wl.make_weights(shape, 77)
    hs = wl.HiddenStream(shape, 77)
    xs = [hs.first()] + [hs.advance(wl.uniform_positions(hs.rng, shape, changed)) for _ in modes]
    outs = []
    for rep in range(2):
        g = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
        ys = [g.step(parity.to_device(xs[0], shape), 3, 0.1).clone()]
        for x, mode in zip(xs[1:], modes):
            ys.append(g.step(parity.to_device(x, shape), mode, 0.1).clone())
        torch.cuda.synchronize()
        c = g.read_caches(shape.batch, shape.seq)
        outs.append((ys, c))
        g.close()
    for a, b in zip(outs[0][0], outs[1][0]):
        assert torch.equal(a, b)
    for k in ("k", "v", "o", "q_prev"):
        np.testing.assert_array_equal(outs[0][1][k], outs[1][1][k])


@pytest.mark.parametrize("mode", ["both", "kv", "o", "dense"])
def test_step_replays_from_a_cuda_graph(dare, mode):
    """A reuse step captured once into a CUDA graph (programmatic launch edges included) and replayed with new inputs
    in the same buffers gives, replay after replay, bit for bit what the same steps give when enqueued one by one: the
    step takes every data-dependent decision on the device and makes no call that a capture forbids."""
    import torch
    shape = wl.scaled(wl.LLADA_LAYER, d_model=512, n_heads=4, batch=2, seq=320, prompt=160)
    w = wl.make_weights(shape, 31)
    hs = wl.HiddenStream(shape, 31)
    eager = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    graphed = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    xs = [hs.first()] + [hs.advance(wl.uniform_positions(hs.rng, shape, n)) for n in (40, 0, 150, 320, 17)]
    xd = [parity.to_device(x, shape) for x in xs]
    m = MODES[mode]
    x_buf, y_buf = torch.empty_like(xd[0]), torch.empty_like(xd[0])
    # first step (dense, fills the caches) and one reuse step outside the graph: the captured step then meets the
    # same host-side state on every replay
    for l in (eager, graphed):
        l.step(xd[0], m, 0.1)
        l.step(xd[1], m, 0.1)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.graph(graph, stream=side):
        graphed.step(x_buf, m, 0.1, y=y_buf)
    for t in range(2, len(xd)):
        x_buf.copy_(xd[t])
        graph.replay()
        ye = eager.step(xd[t], m, 0.1)
        torch.cuda.synchronize()
        assert torch.equal(ye, y_buf), (mode, t)
        if mode != "dense":
            se, sg = eager.last_selection(2, 320), graphed.last_selection(2, 320)
            np.testing.assert_array_equal(se["idx"], sg["idx"])
            np.testing.assert_array_equal(se["delta"], sg["delta"])
    for l in (eager, graphed):
        assert l.status() == 0
        l.close()


def test_selection_across_chunks_and_threshold_extremes(dare):
    """5700 tokens (three sequences of 1900): the selection launch has two CTAs, the second one starting its part of
    the list at the first one's count.  Ordinary threshold, a negative one (everything refreshed) and +inf (nothing)."""
    shape = wl.scaled(wl.LLADA_LAYER, d_model=256, n_heads=2, batch=3, seq=1900, prompt=900)
    w = wl.make_weights(shape, 41)
    hs = wl.HiddenStream(shape, 41)
    g = dare.Layer(shape, w, kernel_path=dare.PATH_TENSOR)
    o = parity.oracle_layer(shape, w)
    parity.compare_step(g, o, hs.first(), 3, 0.1, shape, first=True)
    for n, tau in ((300, 0.1), (40, -1.0), (500, float("inf")), (1900, 0.1), (0, 0.1)):
        ch = wl.uniform_positions(hs.rng, shape, n)
        parity.compare_step(g, o, hs.advance(ch), 3, tau, shape)
        sel = g.last_selection(3, 1900)
        if tau == 0.1:
            np.testing.assert_array_equal(sel["idx"], np.nonzero(ch.reshape(-1))[0])
        elif tau < 0:
            assert sel["count"] == 5700
        else:
            assert sel["count"] == 0
    assert g.status() == 0
    g.close()
