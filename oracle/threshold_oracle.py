"""Plain-loop restatement of the layer-wise threshold allocation of Sec. 3.1 (TEST INFRASTRUCTURE ONLY).

s_l = E_{t,i} s(q_t, q_{t-1}) (Eq. 1); phi_l = L phi_bar softmax(-s_l / eps) (clipped to [0, 1] where the paper is
silent); tau_l = phi_l-quantile of the layer's scores, taken as the linear interpolation between the two order
statistics around position phi_l (n - 1).
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
