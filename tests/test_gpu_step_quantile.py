"""The step that takes its threshold from its own scores (tau_t = the k-th smallest drift score of the step, found on
the device) against the oracle: the order statistic is the plain sort-and-index of oracle/threshold_oracle.py on the
oracle's scores, the step itself is the ordinary oracle step at that threshold."""
import copy

import numpy as np
import pytest

from oracle import dare_oracle as orc
from oracle import threshold_oracle as tor
from paper_2605_08134_b200 import workloads as wl
from tests import parity, rounding

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dare():
    from paper_2605_08134_b200 import build
    build.build()
    from paper_2605_08134_b200 import dare as d
    return d


def test_kth_score_is_the_order_statistic(dare):
    """Stand-alone selection on raw score arrays: bit-exact against sort-and-index, with ties, negative zeros, NaN and
    infinities in the array, for k from 0 to n."""
    import torch
    rng = np.random.default_rng(12)
    stream = torch.cuda.current_stream().cuda_stream
    for n in (1, 5, 1000, 4097, 70_001):
        s = (rng.random(n) ** 6).astype(np.float32)
        s[rng.random(n) < 0.3] = np.float32(3e-6)                     # many ties
        if n > 4:
            s[1], s[2], s[3] = np.float32(-1e-7), np.float32(np.inf), np.float32(-0.0)
        if n > 100:
            s[rng.integers(0, n, 7)] = np.nan
        sd = torch.from_numpy(s).cuda()
        out = torch.zeros(1, device="cuda")
        n_num = int(np.sum(~np.isnan(s)))
        for k in sorted({0, 1, 2, n // 3, n // 2, n_num - 1, n_num, n_num + 1, n - 1, n, n + 5}):
            if k < 0:
                continue
            assert dare.dare_score_kth(sd.data_ptr(), n, k, out.data_ptr(), stream) == 0
            torch.cuda.synchronize()
            want = np.float32(tor.step_threshold(s.tolist(), min(k, n)))
            got = out.cpu().numpy()[0]
            assert got == want or (np.isnan(got) and np.isnan(want)), (n, k, got, want)
            assert np.signbit(got) == np.signbit(want) or got != 0.0
    small = torch.zeros(4, device="cuda")
    assert dare.dare_score_kth(small.data_ptr(), 0, 1, small.data_ptr(), stream) == dare.ERR_SHAPE
    assert dare.dare_score_kth(0, 4, 1, small.data_ptr(), stream) == dare.ERR_INVALID_ARG


CASES = [("fp32-cuda-core", wl.TINY_F32, "simt"),
         ("bf16-tensor", wl.scaled(wl.LLADA_LAYER, d_model=512, n_heads=4, batch=2, seq=320, prompt=160), "tensor"),
         ("bf16-tensor-many-tiles", wl.scaled(wl.LLADA_LAYER, d_model=256, n_heads=2, batch=2, seq=1280, prompt=256), "tensor")]


@pytest.mark.parametrize("name,shape,path", CASES, ids=[c[0] for c in CASES])
def test_step_with_its_own_threshold(dare, name, shape, path):
    """Graded scores (spread over decades).  The reuse counts are chosen where the sorted scores leave a gap of 2e-3 or
    more between the k-th and the (k+1)-th, in the plain fp64 evaluation and in the one with a bf16 x_norm alike: the set
    of the k least-drifted tokens is then the same for every evaluation within 1e-3 of either, the GPU's threshold is its
    own k-th smallest score (within the score gate of the oracle's), and index list, count, offsets, staleness, caches
    and output must agree with the oracle's step at the oracle's threshold."""
    w = wl.make_weights(shape, 88)
    hs = wl.HiddenStream(shape, 88)
    x0 = hs.first()
    x1 = hs.advance_graded(hi=3.0)
    o0 = parity.oracle_layer(shape, w)
    o0.step(x0, 3, 0.1)
    sets = [orc.scores_only(o0, x1)]
    if shape.dtype == wl.DTYPE_BF16:
        r = rounding.rounded_layer(shape, w)
        r.step(x0, 3, 0.1)
        r.step(x1, 0, 0.1)
        sets.append(r.last_scores)
    taus = rounding.clear_thresholds(sets, min_gap=2e-3, limit=4)
    assert len(taus) >= 3
    g = dare.Layer(shape, w, kernel_path={"simt": dare.PATH_SIMT, "tensor": dare.PATH_TENSOR}[path])
    T = shape.tokens
    for i, tau_gap in enumerate(taus):
        k = int((sets[0] < tau_gap).sum())                  # the tokens below the gap: the k least-drifted ones
        assert all(int((s < tau_gap).sum()) == k for s in sets) and 0 < k < T
        tau_o = tor.step_threshold(sets[0].tolist(), k)      # the oracle's order statistic: the largest score below the gap
        assert tau_o < tau_gap and (sets[0] <= tau_o).sum() == k
        mode = (3, 1, 2)[i % 3]
        g.reset()
        g.step(parity.to_device(x0, shape), mode, 0.1)
        yg = g.step_quantile(parity.to_device(x1, shape), mode, k)
        tau_g = g.last_threshold()
        assert abs(tau_g - tau_o) <= parity.SCORE_ATOL[shape.dtype], (tau_g, tau_o)
        o = copy.deepcopy(o0)
        yo = o.step(x1, mode, tau_o)
        sel = g.last_selection(shape.batch, shape.seq)
        assert sel["count"] == T - k
        np.testing.assert_array_equal(sel["idx"], o.last_idx)
        np.testing.assert_array_equal(sel["batch_off"], o.last_batch_off)
        np.testing.assert_array_equal(sel["delta"], o.delta[:shape.batch, :shape.seq])
        assert tau_g == np.sort(sel["scores"])[k - 1]         # the GPU's threshold is its own k-th smallest score
        tol = parity.tol_of(shape.dtype)
        parity.assert_close("y", yg.float().cpu().numpy(), yo, tol, rel_rms=tol)
        c = g.read_caches(shape.batch, shape.seq)
        mf = 2.0 if shape.dtype == wl.DTYPE_BF16 else 1.0
        parity.assert_close("k_cache", c["k"], o.k_cache, tol, max_factor=mf)
        parity.assert_close("o_cache", c["o"], o.o_cache, tol, max_factor=mf)
    # the extremes, and what a first step and the dense mode do with a count
    for k, want in ((0, T), (T, 0), (T + 7, 0)):
        g.reset()
        g.step_quantile(parity.to_device(x0, shape), 3, k)    # first step: dense whatever the count
        assert g.last_selection(shape.batch, shape.seq)["count"] == T
        g.step_quantile(parity.to_device(x1, shape), 3, k)
        assert g.last_selection(shape.batch, shape.seq)["count"] == want
        assert g.last_threshold() == (-np.inf if k == 0 else np.inf)
    g.step_quantile(parity.to_device(x1, shape), 0, 5)
    assert g.last_selection(shape.batch, shape.seq)["count"] == T
    g.step(parity.to_device(x1, shape), 3, 0.25)
    assert g.last_threshold() == 0.25                          # a caller's threshold is reported as given
    with pytest.raises(dare.DareError):
        g.step_quantile(parity.to_device(x1, shape), 3, -1)
    assert g.status() == 0
    g.close()
