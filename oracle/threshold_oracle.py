"""Plain-loop restatement of the layer-wise threshold allocation of Sec. 3.1 (TEST INFRASTRUCTURE ONLY).

s_l = E_{t,i} s(q_t, q_{t-1}) (Eq. 1); phi_l = L phi_bar softmax(-s_l / eps) (clipped to [0, 1] where the paper is
silent); tau_l = phi_l-quantile of the layer's scores, taken as the linear interpolation between the two order
statistics around position phi_l (n - 1).

Per-step form (`step_threshold`): the same quantile taken over the scores of one denoising step, as an order statistic:
tau_t = the k-th smallest score, so that under Eq. 2 (reuse iff s <= tau) the k tokens that drifted least are reused,
and every token tied with the k-th.
"""
import math


def allocate(samples, phi_bar, eps):
    L = len(samples)
    s = [sum(float(v) for v in x) / len(x) for x in samples]
    m = max(-v / eps for v in s)
    e = [math.exp(-v / eps - m) for v in s]
    z = sum(e)
    phi = [min(1.0, max(0.0, L * phi_bar * v / z)) for v in e]
    tau = []
    for x, p in zip(samples, phi):
        xs = sorted(float(v) for v in x)
        pos = p * (len(xs) - 1)
        lo = int(math.floor(pos))
        hi = min(lo + 1, len(xs) - 1)
        tau.append(xs[lo] + (xs[hi] - xs[lo]) * (pos - lo))
    return tau, phi, s


def step_threshold(scores, reuse_count):
    """tau_t = the reuse_count-th smallest of the step's drift scores (plain sort, then index).

    reuse_count <= 0: -inf (no score is <= tau: every token is refreshed).  reuse_count >= number of tokens: +inf.  NaN
    scores are not numbers to compare: they are left out of the sort (such tokens are refreshed whatever tau is), and a
    reuse_count beyond the scores that remain gives +inf."""
    n = len(scores)
    if reuse_count <= 0:
        return -math.inf
    if reuse_count >= n:
        return math.inf
    finite_or_inf = []
    for v in scores:
        v = float(v)
        if v == v:
            finite_or_inf.append(v)
    if reuse_count > len(finite_or_inf):
        return math.inf
    finite_or_inf.sort()
    return finite_or_inf[reuse_count - 1]
