"""GPU parity of the CUDA-core kernel path against the fp64 oracle (element by element, same seeded inputs)."""
import numpy as np
import pytest

from paper_2605_08134_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

MODES = {"kv": 1, "o": 2, "both": 3, "dense": 0}


@pytest.fixture(scope="module")
def dare():
    from paper_2605_08134_b200 import build
    build.build()
    from paper_2605_08134_b200 import dare as d
    return d


@pytest.mark.parametrize("mode", list(MODES))
def test_config1_tiny_fp32_two_steps(dare, mode):
    """Config 1: d=256, 4 heads x 64, seq 128, fp32; step 0 (dense) then step 1 with 20 % of tokens redrawn."""
    shape = wl.TINY_F32
    w, x0, x1, changed = wl.two_step_case(shape, 26)
    g = dare.Layer(shape, w)
    o = parity.oracle_layer(shape, w)
    parity.compare_step(g, o, x0, MODES[mode], 0.1, shape, first=True)
    assert g.launch_count() > 0
    parity.compare_step(g, o, x1, MODES[mode], 0.1, shape)
    sel = g.last_selection(shape.batch, shape.seq)
    if mode != "dense":
        np.testing.assert_array_equal(sel["idx"], np.nonzero(changed.reshape(-1))[0])
    else:
        assert sel["count"] == shape.tokens
    g.close()


@pytest.mark.parametrize("mode", ["kv", "o", "both"])
def test_reused_rows_are_bit_identical(dare, mode):
    """Eq. 3 / Eq. 4: rows of the reuse set are not touched by the step."""
    shape = wl.TINY_F32
    w, x0, x1, changed = wl.two_step_case(shape, 26)
    g = dare.Layer(shape, w)
    g.step(parity.to_device(x0, shape), MODES[mode], 0.1)
    before = g.read_caches(1, shape.seq)
    g.step(parity.to_device(x1, shape), MODES[mode], 0.1)
    after = g.read_caches(1, shape.seq)
    keep = ~changed
    if MODES[mode] & 1:
        assert np.array_equal(after["k"][keep], before["k"][keep]) and np.array_equal(after["v"][keep], before["v"][keep])
    if MODES[mode] & 2:
        assert np.array_equal(after["o"][keep], before["o"][keep])
    assert not np.array_equal(after["o"][changed], before["o"][changed])
    g.close()


@pytest.mark.parametrize("mode", ["kv", "o", "both"])
def test_thresholds_at_the_extremes(dare, mode):
    shape = wl.TINY_F32
    w, x0, x1, _ = wl.two_step_case(shape, 26)
    for tau, expect in ((-1.0, shape.tokens), (0.0, shape.tokens), (float("inf"), 0)):
        g = dare.Layer(shape, w)
        o = parity.oracle_layer(shape, w)
        parity.compare_step(g, o, x0, MODES[mode], tau, shape, first=True)
        # tau = 0 sits inside the cloud of near-zero scores: compare without the margin rule, counts only
        yg = g.step(parity.to_device(x1, shape), MODES[mode], tau)
        yo = o.step(x1, MODES[mode], tau)
        sel = g.last_selection(1, shape.seq)
        if tau != 0.0:
            assert sel["count"] == expect == len(o.last_idx)
            parity.assert_close("y", yg.float().cpu().numpy(), yo, parity.TOL_F32)
        else:
            assert sel["count"] >= shape.tokens - 2      # fp32 may round a 1e-7 score to exactly 0
        g.close()


def test_multi_step_batched_ragged_simt(dare):
    """Batch 3, seq 80 (not a multiple of any tile), 5 steps, mode both; bf16 storage on the CUDA-core path."""
    for dtype in (wl.DTYPE_F32, wl.DTYPE_BF16):
        shape = wl.scaled(wl.TINY_F32, batch=3, seq=80, prompt=40, dtype=dtype, d_model=128, n_heads=4, head_dim=32)
        w = wl.make_weights(shape, 5)
        hs = wl.HiddenStream(shape, 5)
        g = dare.Layer(shape, w, kernel_path=dare.PATH_SIMT)
        o = parity.oracle_layer(shape, w)
        parity.compare_step(g, o, hs.first(), 3, 0.1, shape, first=True)
        for t in range(4):
            ch = wl.uniform_positions(hs.rng, shape, 9)
            parity.compare_step(g, o, hs.advance(ch), (3, 1, 2, 3)[t], 0.1, shape)
        g.close()


def test_window_steps_keep_the_prefix(dare):
    """Steps over a generation window [p, S): prompt rows of every cache stay frozen (prefix cache)."""
    shape = wl.scaled(wl.TINY_F32, batch=2, seq=96, prompt=40)
    w = wl.make_weights(shape, 6)
    hs = wl.HiddenStream(shape, 6)
    g = dare.Layer(shape, w)
    o = parity.oracle_layer(shape, w)
    parity.compare_step(g, o, hs.first(), 3, 0.1, shape, first=True)
    p = shape.prompt
    for t in range(3):
        ch = wl.uniform_positions(hs.rng, shape, 12)
        x = hs.advance(ch)
        parity.compare_step(g, o, np.ascontiguousarray(x[:, p:]), 3, 0.1, shape, pos_begin=p)
    g.close()


def test_reset_and_state_rules(dare):
    shape = wl.TINY_F32
    w, x0, x1, _ = wl.two_step_case(shape, 26)
    g = dare.Layer(shape, w, max_batch=2)
    o = parity.oracle_layer(shape, w, max_batch=2)
    xd = parity.to_device(x0, shape)
    # first step must start at position 0
    with pytest.raises(dare.DareError) as e:
        g.step(xd[:, 64:].contiguous(), 3, 0.1, pos_begin=64)
    assert e.value.status == dare.ERR_STATE
    parity.compare_step(g, o, x0, 3, 0.1, shape, first=True)
    # batch change without reset
    import torch
    with pytest.raises(dare.DareError) as e:
        g.step(torch.cat([xd, xd]), 3, 0.1)
    assert e.value.status == dare.ERR_STATE
    with pytest.raises(dare.DareError) as e:
        g.step(xd, 3, float("nan"))
    assert e.value.status == dare.ERR_INVALID_ARG
    with pytest.raises(dare.DareError) as e:
        g.step(xd, 4, 0.1)
    assert e.value.status == dare.ERR_INVALID_ARG
    # reset: next step is dense again and matches a fresh oracle
    g.reset(); o.reset()
    parity.compare_step(g, o, x1, 3, 0.1, shape, first=True)
    parity.compare_step(g, o, x0, 3, 0.1, shape)
    g.close()


def test_export_import_state_roundtrip(dare):
    import torch
    shape = wl.TINY_F32
    w, x0, x1, _ = wl.two_step_case(shape, 26)
    a = dare.Layer(shape, w)
    b = dare.Layer(shape, w)
    a.step(parity.to_device(x0, shape), 3, 0.1)
    n = dare.dare_layer_state_bytes(a.handle)
    blob = torch.empty(n, dtype=torch.uint8).pin_memory()
    assert dare.dare_layer_export_state(a.handle, blob.data_ptr(), n) == 0
    assert dare.dare_layer_export_state(a.handle, blob.data_ptr(), n - 1) == dare.ERR_WORKSPACE
    assert dare.dare_layer_import_state(b.handle, blob.data_ptr(), n) == 0
    ya = a.step(parity.to_device(x1, shape), 3, 0.1)
    yb = b.step(parity.to_device(x1, shape), 3, 0.1)
    torch.cuda.synchronize()
    assert torch.equal(ya, yb)
    assert np.array_equal(a.last_selection(1, 128)["idx"], b.last_selection(1, 128)["idx"])
    a.close(); b.close()


def test_step_host_matches_device_step(dare):
    import torch
    shape = wl.TINY_F32
    w, x0, x1, _ = wl.two_step_case(shape, 26)
    a = dare.Layer(shape, w)
    b = dare.Layer(shape, w)
    for x in (x0, x1):
        xh = torch.from_numpy(x).pin_memory()
        yh = torch.empty_like(xh).pin_memory()
        b.step_host(xh, 3, 0.1, yh)
        ya = a.step(parity.to_device(x, shape), 3, 0.1)
        torch.cuda.synchronize()
        assert torch.equal(ya.cpu(), yh)
    a.close(); b.close()


def test_step_host_async_pipeline_matches_device_steps(dare):
    """Four layers stepped through the enqueue-only host-buffer entry point, three rounds without waiting in between
    (copies of one layer overlap kernels of another; a layer's staging buffers are reused from round to round), against
    the same steps with device buffers: bit-identical outputs."""
    import torch
    shape = wl.TINY_F32
    w, x0, x1, _ = wl.two_step_case(shape, 26)
    n = 4
    ref = [dare.Layer(shape, w) for _ in range(n)]
    pipe = [dare.Layer(shape, w) for _ in range(n)]
    xs = [x0, x1, x0]
    xh = [[torch.from_numpy(np.ascontiguousarray(x + 0.01 * i)).pin_memory() for x in xs] for i in range(n)]
    yh = [[torch.empty_like(xh[i][r]).pin_memory() for r in range(len(xs))] for i in range(n)]
    for r in range(len(xs)):
        for i in range(n):
            pipe[i].step_host_async(xh[i][r], 3, 0.1, yh[i][r])
    for i in range(n):
        pipe[i].wait_host()
    for r in range(len(xs)):
        for i in range(n):
            ya = ref[i].step(xh[i][r].cuda(), 3, 0.1)
            torch.cuda.synchronize()
            assert torch.equal(ya.cpu(), yh[i][r]), (r, i)
    for l in ref + pipe:
        assert l.status() == 0
        l.close()
