"""Index sets next to the threshold (GPU).  The other workloads are bimodal (reused tokens score ~1e-6, redrawn ones
~1, tau = 0.1), so their index-set checks would survive a score error of several 1e-2.  Here every token gets noise
whose size is drawn log-uniformly, the scores spread over decades, and the thresholds sit in gaps of the sorted scores
only 2e-3 wide: every score is at least 1e-3 away from tau, as the bit-exact index-set check requires, and a GPU score
that is off by much more than that puts a token on the wrong side of some threshold.  For the bf16 path the gaps are
clear of two evaluations: the plain fp64 oracle and the fp64 evaluation with x_norm rounded to bf16, which is what the
kernels score."""
import copy

import numpy as np
import pytest

from oracle import dare_oracle as orc
from paper_2605_08134_b200 import workloads as wl
from tests import parity, rounding

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dare():
    from paper_2605_08134_b200 import build
    build.build()
    from paper_2605_08134_b200 import dare as d
    return d


TINY = wl.TINY_F32
SMALL_BF16 = wl.scaled(wl.LLADA_LAYER, d_model=512, n_heads=4, batch=2, seq=320, prompt=160)
PAIR_BF16 = wl.scaled(wl.LLADA_LAYER, d_model=1024, n_heads=8, batch=1, seq=256, prompt=128)   # two row tiles: narrow MMA pairs
CASES = [
    ("fp32-cuda-core", TINY, "simt", 0), ("fp32-cuda-core-head3", TINY, "simt", 3),
    ("bf16-tensor", SMALL_BF16, "tensor", 0), ("bf16-tensor-head1", SMALL_BF16, "tensor", 1),
    ("bf16-tensor-head2", SMALL_BF16, "tensor", 2), ("bf16-tensor-pairs-head5", PAIR_BF16, "tensor", 5),
    ("bf16-cuda-core-head1", SMALL_BF16, "simt", 1),
]


@pytest.mark.parametrize("name,shape,path,score_head", CASES, ids=[c[0] for c in CASES])
def test_index_sets_at_thresholds_inside_narrow_score_gaps(dare, name, shape, path, score_head):
    w = wl.make_weights(shape, 77)
    hs = wl.HiddenStream(shape, 77)
    x0 = hs.first()
    x1 = hs.advance_graded(hi=3.0)
    o0 = parity.oracle_layer(shape, w, score_head=score_head)
    o0.step(x0, 3, 0.1)
    sets = [orc.scores_only(o0, x1)]
    if shape.dtype == wl.DTYPE_BF16:
        r = rounding.rounded_layer(shape, w, score_head=score_head)
        r.step(x0, 3, 0.1)
        r.step(x1, 0, 0.1)
        sets.append(r.last_scores)
    assert sets[0].min() < 1e-4 and sets[0].max() > 0.2                 # scores spread over decades
    taus = rounding.clear_thresholds(sets, min_gap=2e-3, limit=6)
    assert len(taus) >= 3, taus
    assert max(taus) > 3 * min(taus)                                    # thresholds over a range of the distribution
    g = dare.Layer(shape, w, kernel_path={"simt": dare.PATH_SIMT, "tensor": dare.PATH_TENSOR}[path],
                   score_head=score_head)
    counts = []
    for i, tau in enumerate(taus):
        mode = (3, 1, 2)[i % 3]
        g.reset()
        g.step(parity.to_device(x0, shape), mode, tau)
        o = copy.deepcopy(o0)
        parity.compare_step(g, o, x1, mode, tau, shape)                 # list, count, offsets, staleness: bit-exact
        counts.append(len(o.last_idx))
        for s in sets:                                                  # the gap really is clear, in both evaluations
            assert np.abs(s - tau).min() >= parity.MARGIN
        assert np.abs(sets[0] - tau).min() < 3.5e-3                     # ... and narrow: a score within 3.5e-3 of tau
    assert len(set(counts)) == len(counts) and 0 < min(counts) and max(counts) < shape.tokens
    g.close()
