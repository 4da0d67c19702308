"""The device-reported error paths, without faulting, trapping or hanging the device: a bounded wait that runs out
(a one-CTA launch waits, with a limit of a millisecond, on a barrier nothing arrives on) and range checks on the
device-side selection (a step whose refresh list or list length is overwritten with a value just outside the step: the
kernels must record it, skip the access that would have used it, and finish normally)."""
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


SMALL_BF16 = wl.scaled(wl.LLADA_LAYER, d_model=512, n_heads=4, batch=2, seq=320, prompt=160)
MANY_TILES = wl.scaled(wl.LLADA_LAYER, d_model=256, n_heads=2, batch=2, seq=1280, prompt=256)   # persistent, listed launches


def _two_steps_ok(dare, g, o, hs, shape, mode=3):
    """An ordinary reuse step on the handle, compared with the oracle in full."""
    ch = wl.uniform_positions(hs.rng, shape, 37)
    parity.compare_step(g, o, hs.advance(ch), mode, 0.1, shape)


@pytest.mark.parametrize("path", ["tensor", "simt"])
def test_bounded_wait_runs_out_and_the_handle_recovers(dare, path):
    shape = SMALL_BF16
    w = wl.make_weights(shape, 5)
    hs = wl.HiddenStream(shape, 5)
    g = dare.Layer(shape, w, kernel_path={"tensor": dare.PATH_TENSOR, "simt": dare.PATH_SIMT}[path])
    o = parity.oracle_layer(shape, w)
    parity.compare_step(g, o, hs.first(), 3, 0.1, shape, first=True)
    assert g.status() == dare.OK
    waited = g.wait_probe(1_000_000)                      # 1 ms
    assert 1_000_000 <= waited < 50_000_000, waited        # gave up after the limit, within milliseconds
    assert g.status() == dare.ERR_TIMEOUT
    assert g.status() == dare.ERR_TIMEOUT                  # the first error stays ...
    waited2 = g.wait_probe(1_000_000)
    assert waited2 < 1_000_000                             # ... and while it stands a wait gives up at once
    g.clear_status()
    assert g.status() == dare.OK
    _two_steps_ok(dare, g, o, hs, shape)                   # same handle, same caches: the next step is right
    assert g.status() == dare.OK
    g.close()


@pytest.mark.parametrize("case", ["tensor-short", "tensor-many-tiles", "simt"])
@pytest.mark.parametrize("what", [1, 2])
def test_selection_values_out_of_range_are_flagged_and_skipped(dare, case, what):
    shape = MANY_TILES if case == "tensor-many-tiles" else SMALL_BF16
    path = dare.PATH_SIMT if case == "simt" else dare.PATH_TENSOR
    w = wl.make_weights(shape, 9)
    hs = wl.HiddenStream(shape, 9)
    g = dare.Layer(shape, w, kernel_path=path)
    o = parity.oracle_layer(shape, w)
    parity.compare_step(g, o, hs.first(), 3, 0.1, shape, first=True)
    _two_steps_ok(dare, g, o, hs, shape)
    before = g.read_caches(shape.batch, shape.seq)
    ch = wl.uniform_positions(hs.rng, shape, 41)
    x = hs.advance(ch)
    g.inject(what)
    y = g.step(parity.to_device(x, shape), 3, 0.1)
    assert g.status() == dare.ERR_DEVICE_CHECK
    after = g.read_caches(shape.batch, shape.seq)
    planned = np.nonzero(ch.reshape(-1))[0]
    yh = y.float().cpu().numpy().reshape(shape.tokens, -1)
    assert np.isfinite(np.delete(yh, planned[0], axis=0)).all()      # (the skipped row of y is whatever the buffer held)
    if what == 1:
        # the overwritten entry named no token of the step: its row was skipped, every other refreshed row was written,
        # rows outside the refresh set are untouched
        first = planned[0]
        b, i = divmod(int(first), shape.seq)
        assert np.array_equal(after["k"][b, i], before["k"][b, i]) and np.array_equal(after["o"][b, i], before["o"][b, i])
        rest = planned[1:]
        rb, ri = rest // shape.seq, rest % shape.seq
        assert not np.array_equal(after["k"][rb, ri], before["k"][rb, ri])
        keep = ~ch
        assert np.array_equal(after["k"][keep], before["k"][keep]) and np.array_equal(after["o"][keep], before["o"][keep])
    # (what = 2: the list's length is clamped to the step's tokens, so entries past the true end, left by earlier steps,
    # are processed as well: valid tokens, refreshed needlessly; nothing is read or written outside the step)
    # the handle recovers: clear the status, forget the half-written caches, and it agrees with the oracle again
    g.clear_status()
    g.reset(); o.reset()
    parity.compare_step(g, o, x, 3, 0.1, shape, first=True)
    _two_steps_ok(dare, g, o, hs, shape)
    assert g.status() == dare.OK
    g.close()
