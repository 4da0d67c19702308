"""Stand-alone drift score and multi-tile compaction at token counts far beyond one layer step, against the oracle."""
import numpy as np
import pytest

from oracle import dare_oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dare():
    from paper_2605_08134_b200 import build
    build.build()
    from paper_2605_08134_b200 import dare as d
    return d


def _scores(n, seed):
    """Bimodal scores like the method's: most tokens near zero, a fraction spread over (0.3, 1.5); some NaN, +-inf."""
    rng = np.random.default_rng(seed)
    s = np.abs(rng.standard_normal(n).astype(np.float32)) * np.float32(1e-5)
    hot = rng.random(n) < 0.13
    s[hot] = rng.uniform(0.3, 1.5, int(hot.sum())).astype(np.float32)
    if n > 10:
        s[3] = np.nan; s[7] = np.inf; s[9] = -np.inf
    return s


@pytest.mark.parametrize("n", [0, 1, 2, 3, 5, 4095, 4096, 4097, 16383, 16384, 16385, 16387, 100_003, 1 << 20, (1 << 22) + 12345, (1 << 24) + 20_000])
def test_select_compact_matches_the_predicate(dare, n):
    import torch
    s = _scores(n, n % 97)
    sd = torch.from_numpy(s).cuda() if n else torch.zeros(4, device="cuda")
    idx = torch.full((max(n, 1),), -1, dtype=torch.int32, device="cuda")
    cnt = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    nb = dare.dare_select_compact_scratch_bytes(n)
    assert nb >= 256
    scratch = torch.empty(nb, dtype=torch.uint8, device="cuda")
    for tau in (0.1, -1.0, float("inf")):
        st = dare.dare_select_compact(sd.data_ptr(), n, tau, idx.data_ptr(), cnt.data_ptr(), scratch.data_ptr(), nb,
                                      torch.cuda.current_stream().cuda_stream)
        assert st == 0
        torch.cuda.synchronize()
        want = np.nonzero(orc.refresh_mask(s, tau))[0]
        assert int(cnt.item()) == len(want)
        np.testing.assert_array_equal(idx[:len(want)].cpu().numpy(), want)


def test_select_compact_rejects_bad_arguments(dare):
    import torch
    sd = torch.zeros(1024, device="cuda")
    idx = torch.zeros(1024, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(1, dtype=torch.int32, device="cuda")
    scratch = torch.empty(4096, dtype=torch.uint8, device="cuda")
    ok = (sd.data_ptr(), 1024, 0.1, idx.data_ptr(), cnt.data_ptr(), scratch.data_ptr(), 4096)
    assert dare.dare_select_compact(*ok) == 0
    assert dare.dare_select_compact(0, *ok[1:]) == dare.ERR_INVALID_ARG
    assert dare.dare_select_compact(ok[0], 1024, float("nan"), *ok[3:]) == dare.ERR_INVALID_ARG
    assert dare.dare_select_compact(ok[0], -1, *ok[2:]) == dare.ERR_SHAPE
    assert dare.dare_select_compact(*ok[:6], 16) == dare.ERR_WORKSPACE
    assert dare.dare_select_compact(ok[0] + 4, *ok[1:]) == dare.ERR_ALIGN
    assert dare.dare_select_compact_scratch_bytes(-5) == 0


@pytest.mark.parametrize("rows,hd", [(1, 128), (1000, 64), (65537, 128)])
def test_drift_scores_match_oracle(dare, rows, hd):
    import torch
    rng = np.random.default_rng(rows)
    a = rng.standard_normal((rows, hd)).astype(np.float32)
    b = (a + 0.3 * rng.standard_normal((rows, hd))).astype(np.float32)
    b[0] = 0.0                                     # zero-norm row: score 1
    if rows > 2:
        b[1] = a[1]; b[2] = -a[2]
    ad, bd = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
    out = torch.empty(rows, device="cuda")
    assert dare.dare_drift_scores(ad.data_ptr(), bd.data_ptr(), rows, hd, out.data_ptr()) == 0
    torch.cuda.synchronize()
    want = orc.drift_score(a, b)
    np.testing.assert_allclose(out.cpu().numpy(), want, rtol=0, atol=2e-6)
    assert out[0].item() == 1.0
    assert dare.dare_drift_scores(ad.data_ptr(), bd.data_ptr(), rows, 6, out.data_ptr()) == dare.ERR_SHAPE


@pytest.mark.parametrize("n", [300_000, (1 << 24) + 20_000])
def test_select_compact_alternating_thresholds_on_one_scratch(dare, n):
    """Calls in a row on the same scratch whose decisions differ completely (nothing refreshed, then the ordinary set,
    then everything): a pass that read what an earlier call left at the same addresses would show here."""
    import torch
    s = _scores(n, 5)
    sd = torch.from_numpy(s).cuda()
    idx = torch.empty(n, dtype=torch.int32, device="cuda")
    cnt = torch.empty(1, dtype=torch.int32, device="cuda")
    nb = dare.dare_select_compact_scratch_bytes(n)
    scratch = torch.zeros(nb, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    want = {tau: np.nonzero(orc.refresh_mask(s, tau))[0] for tau in (float("inf"), 0.1, -1.0)}
    for rep in range(4):
        for tau in (float("inf"), 0.1, -1.0):
            idx.fill_(-1)
            assert dare.dare_select_compact(sd.data_ptr(), n, tau, idx.data_ptr(), cnt.data_ptr(), scratch.data_ptr(),
                                            nb, stream) == 0
            torch.cuda.synchronize()
            k = int(cnt.item())
            assert k == len(want[tau]), (rep, tau)
            assert np.array_equal(idx[:k].cpu().numpy(), want[tau]), (rep, tau)
            assert bool((idx[k:] == -1).all())


@pytest.mark.parametrize("rows,d,dtype", [(7, 256, "f32"), (300, 1024, "bf16"), (2049, 4096, "bf16"), (4100, 512, "bf16"),
                                          (5000, 768, "f32")])
def test_standalone_rmsnorm_matches_the_oracle(dare, rows, d, dtype):
    """Alg. 1/2 line 1 through its own entry point, on both of its kernels (one row per CTA; two rows per CTA beyond 2048
    bf16 rows), with a gain that is not all ones."""
    import torch
    from oracle import dare_oracle as orc
    from paper_2605_08134_b200 import workloads as wl
    rng = np.random.default_rng(rows + d)
    bf = dtype == "bf16"
    x = wl.round_to(rng.standard_normal((rows, d), dtype=np.float32) * 1.7, wl.DTYPE_BF16 if bf else wl.DTYPE_F32)
    gain = (1.0 + 0.2 * rng.standard_normal(d)).astype(np.float32)
    tdt = torch.bfloat16 if bf else torch.float32
    xd = torch.from_numpy(x).cuda().to(tdt)
    gd = torch.from_numpy(gain).cuda()
    yd = torch.empty_like(xd)
    st = dare.dare_rmsnorm(xd.data_ptr(), gd.data_ptr(), yd.data_ptr(), rows, d, 1e-5, dare.BF16 if bf else dare.F32,
                           torch.cuda.current_stream().cuda_stream)
    assert st == 0
    torch.cuda.synchronize()
    want = orc.rmsnorm(x, gain, 1e-5)
    got = yd.float().cpu().numpy().astype(np.float64)
    # bf16: one rounding of the result (relative 2^-9); fp32: fp32 arithmetic on O(1) values
    tol = 2.0 ** -8 if bf else 2e-6
    assert np.max(np.abs(got - want) / (np.abs(want) + 1.0)) <= tol
    assert dare.dare_rmsnorm(0, gd.data_ptr(), yd.data_ptr(), rows, d, 1e-5, dare.F32, 0) == dare.ERR_INVALID_ARG
    assert dare.dare_rmsnorm(xd.data_ptr(), gd.data_ptr(), yd.data_ptr(), rows, d + 1, 1e-5, dare.F32, 0) == dare.ERR_SHAPE
