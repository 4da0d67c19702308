"""The compaction entry point for callers that cannot allocate device memory (a server whose arena owns all of HBM,
or a loop that cannot afford cudaMalloc's device-wide synchronisation): its scratch is a fixed array inside the
library.  Checked against the entry point that takes caller scratch, on calls in a row: the second smaller than the
first, so that the array still holds the first call's tile counts beyond the second call's range, the third as large as
the array allows.

Collected last on purpose: a failure here must not hide any other test from a run that stops at the first failure.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _scores(n, seed):
    rng = np.random.default_rng(seed)
    s = np.abs(rng.standard_normal(n).astype(np.float32)) * np.float32(1e-5)
    hot = rng.random(n) < 0.2
    s[hot] = rng.uniform(0.3, 1.5, int(hot.sum())).astype(np.float32)
    return s


def test_static_scratch_variant_matches_caller_scratch_variant_twice_in_a_row():
    import torch
    from paper_2605_08134_b200 import build
    build.build()
    from paper_2605_08134_b200 import dare

    stream = torch.cuda.current_stream().cuda_stream
    limit = dare.dare_select_compact_static_max_tokens()
    assert limit == 4096 * 4096
    # (the third call is exactly as large as the built-in array allows: all of its 1024 tiles in use)
    for call, (n, tau, seed) in enumerate([(3_000_017, 0.1, 1), (70_001, 0.5, 2), (limit, 0.1, 3)]):
        s = torch.from_numpy(_scores(n, seed)).cuda()
        idx_a = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        idx_b = torch.full((n,), -2, dtype=torch.int32, device="cuda")
        cnt_a = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        cnt_b = torch.full((1,), -2, dtype=torch.int32, device="cuda")
        nb = dare.dare_select_compact_scratch_bytes(n)
        scratch = torch.empty(nb, dtype=torch.uint8, device="cuda")
        assert dare.dare_select_compact(s.data_ptr(), n, tau, idx_a.data_ptr(), cnt_a.data_ptr(), scratch.data_ptr(), nb,
                                        stream) == 0
        assert dare.dare_select_compact_static(s.data_ptr(), n, tau, idx_b.data_ptr(), cnt_b.data_ptr(), stream) == 0
        torch.cuda.synchronize()
        na, nbk = int(cnt_a.item()), int(cnt_b.item())
        assert na == nbk and 0 < na < n, (call, na, nbk)
        # index work: bit-exact, the tolerance every index comparison in this suite uses
        assert torch.equal(idx_a[:na], idx_b[:na]), f"call {call}: index lists differ"
        assert bool((idx_b[na:] == -2).all())           # nothing written past the list

    # sizes beyond the built-in array are refused, as are the usual bad arguments
    small = torch.zeros(16, device="cuda")
    idx = torch.zeros(16, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = dare.dare_select_compact_static(small.data_ptr(), limit + 1, 0.1, idx.data_ptr(), cnt.data_ptr(), stream)
    assert st == dare.ERR_SHAPE
    assert "shape" in dare.status_string(dare.ERR_SHAPE)
    assert dare.dare_select_compact_static(0, 16, 0.1, idx.data_ptr(), cnt.data_ptr(), stream) == dare.ERR_INVALID_ARG
    st = dare.dare_select_compact_static(small.data_ptr(), 16, float("nan"), idx.data_ptr(), cnt.data_ptr(), stream)
    assert st == dare.ERR_INVALID_ARG
    # and an empty input is a valid call
    assert dare.dare_select_compact_static(small.data_ptr(), 0, 0.1, idx.data_ptr(), cnt.data_ptr(), stream) == 0
    torch.cuda.synchronize()
    assert int(cnt.item()) == 0
