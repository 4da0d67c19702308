"""Layer-wise threshold allocation (Sec. 3.1): the host helper against the plain-loop oracle and its closed forms."""
import numpy as np

from oracle import threshold_oracle as tor
from paper_2605_08134_b200 import thresholds as th


def _samples(L=6, n=500, seed=0):
    rng = np.random.default_rng(seed)
    out = []
    for l in range(L):
        near = np.abs(rng.standard_normal(n)) * 1e-4
        far = rng.uniform(0.2, 1.2, n)
        out.append(np.where(rng.random(n) < 0.5 + 0.07 * l, near, far))     # deeper layers drift less
    return out


def test_matches_plain_loop_oracle():
    smp = _samples()
    for phi_bar, eps in ((0.3, 0.1), (0.5, 0.05), (0.7, 1.0)):
        tau, phi, s = th.thresholds(smp, phi_bar, eps)
        t2, p2, s2 = tor.allocate(smp, phi_bar, eps)
        np.testing.assert_allclose(s, s2, rtol=1e-12)
        np.testing.assert_allclose(phi, p2, rtol=1e-12)
        np.testing.assert_allclose(tau, t2, rtol=1e-10, atol=1e-15)


def test_closed_forms():
    # equal drift everywhere: every layer gets the average quantile
    same = [np.linspace(0, 1, 101)] * 4
    tau, phi, s = th.thresholds(same, 0.3, 0.1)
    np.testing.assert_allclose(phi, 0.3, rtol=1e-12)
    np.testing.assert_allclose(tau, 0.3, rtol=1e-12)          # the 0.3-quantile of a uniform grid on [0, 1]
    # the budget is conserved while no layer saturates: sum phi_l = L * phi_bar
    smp = _samples()
    _, phi, s = th.thresholds(smp, 0.3, 1.0)
    assert phi.max() < 1 and abs(phi.sum() - len(smp) * 0.3) < 1e-12
    # less drift => larger share (softmax of -s)
    assert (np.diff(s) < 0).all() and (np.diff(phi) > 0).all()
    # a sharp temperature saturates the calmest layer at 1: its threshold is its largest score
    tau, phi, _ = th.thresholds(smp, 0.5, 1e-3)
    assert phi[-1] == 1.0 and tau[-1] == smp[-1].max() and phi[0] < 1e-6


def test_thresholds_give_the_planned_reuse_rate():
    """tau_l is a quantile: the share of calibration scores with s <= tau_l is phi_l (Eq. 2 then reuses that share)."""
    smp = _samples(n=4000, seed=3)
    tau, phi, _ = th.thresholds(smp, 0.4, 0.3)
    for x, t, p in zip(smp, tau, phi):
        assert abs(np.mean(x <= t) - p) < 2e-3


# ----------------------------------------------------------------------------- per-step threshold (order statistic)
def test_step_threshold_closed_forms():
    inf = float("inf")
    s = [0.5, 0.1, 0.3, 0.2, 0.4]
    assert tor.step_threshold(s, 0) == -inf and tor.step_threshold(s, -3) == -inf
    assert tor.step_threshold(s, 5) == inf and tor.step_threshold(s, 9) == inf
    assert [tor.step_threshold(s, k) for k in (1, 2, 3, 4)] == [0.1, 0.2, 0.3, 0.4]
    # ties: the threshold is the tied value, and Eq. 2 then reuses every token that has it
    t = [0.3, 0.1, 0.3, 0.3, 0.7]
    assert tor.step_threshold(t, 2) == 0.3 and sum(v <= 0.3 for v in t) == 4
    # negative zero-ish scores (1 - cos rounds below zero) order below positive ones
    assert tor.step_threshold([1e-7, -1e-7, 0.0, 0.5], 1) == -1e-7
    # NaN scores are refreshed whatever the threshold: they are not counted among the reusable ones
    u = [0.2, float("nan"), 0.1, float("nan"), 0.9]
    assert tor.step_threshold(u, 2) == 0.2 and tor.step_threshold(u, 3) == 0.9 and tor.step_threshold(u, 4) == inf
    assert tor.step_threshold([0.2, inf, 0.1], 2) == 0.2


def test_step_threshold_reuses_exactly_the_least_drifted_tokens():
    """Against numpy's partition, and the two counting properties that define an order statistic: fewer than k scores
    lie strictly below tau, at least k lie at or below it; with distinct scores Eq. 2 then reuses exactly k tokens."""
    rng = np.random.default_rng(4)
    for n in (1, 2, 17, 1000):
        s = rng.random(n) ** 4
        for k in sorted({1, n // 3, n // 2, n - 1} - {0, n}):
            tau = tor.step_threshold(s.tolist(), k)
            assert tau == np.partition(s, k - 1)[k - 1]
            assert (s < tau).sum() < k <= (s <= tau).sum()
            assert (s <= tau).sum() == k
    # reuse rate phi -> count floor(phi * n): the quantile form of Sec. 3.1 on one step's scores
    s = np.linspace(0.0, 1.0, 101)
    for phi in (0.0, 0.3, 0.5, 0.87, 1.0):
        k = int(np.floor(phi * len(s) + 1e-9))
        tau = tor.step_threshold(s.tolist(), k)
        assert (s <= tau).sum() == min(k, len(s))
