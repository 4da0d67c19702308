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
