"""The oracle's arithmetic with the storage roundings of the bf16 kernel path put in by hand.

Test infrastructure only.  The fp64 oracle computes on the given inputs without any intermediate rounding; the bf16
kernels keep x_norm, the rotated Q, the cached K, V and the cached attention output in bf16.  `RoundedLayer` takes the
oracle's own functions (rmsnorm, linear, rope, drift_score, refresh_mask, attention_rows) in the oracle's order and
rounds exactly those stored tensors to bf16 (round to nearest even), everything else staying fp64.  It serves three
purposes:
  * it says how far the storage format alone moves scores, caches and outputs away from the plain oracle, which is what
    the tolerances of the bf16 parity tests rest on;
  * it gives the second set of scores that a threshold must stay clear of for the index set of the bf16 path to be
    well defined (the drift score is taken from fp32 accumulators over a bf16 x_norm);
  * it is the comparison for inputs whose logits are so large that the operand rounding, not the kernel, decides the
    distance to the plain oracle.
The stored scoring-head query stays unrounded: the kernels keep it in fp32 from the fp32 accumulators.
"""
from __future__ import annotations

import numpy as np

from oracle import dare_oracle as orc
from paper_2605_08134_b200 import workloads as wl


def r16(a):
    """fp64 array -> nearest bf16 value, returned as fp64."""
    return wl.bf16_round(np.asarray(a, np.float32)).astype(np.float64)


class RoundedLayer(orc.OracleLayer):
    """OracleLayer.step with x_norm, rotated Q, K, V and the attention output rounded to bf16 where the kernels store them."""

    def step(self, x, mode, tau, pos_begin=0):
        x = np.asarray(x, np.float64)
        B, S_act, d = x.shape
        H, hd = self.H, self.hd
        win = slice(pos_begin, pos_begin + S_act)
        T = B * S_act
        positions = np.tile(np.arange(pos_begin, pos_begin + S_act), B)
        xn = r16(orc.rmsnorm(x.reshape(T, d), self.gain, self.eps))
        q = orc.linear(xn, self.w_q)
        q0 = q[:, self.score_head * hd:(self.score_head + 1) * hd]
        scores = orc.drift_score(q0, self.q_prev[:B, win].reshape(T, hd)) if self.has_prev else np.full(T, np.inf)
        sel = np.ones(T, bool) if (mode == orc.MODE_DENSE or not self.has_prev) else orc.refresh_mask(scores, tau)
        idx = np.nonzero(sel)[0]
        self.q_prev[:B, win] = q0.reshape(B, S_act, hd)
        kv_rows = idx if (mode & orc.MODE_KV) else np.arange(T)
        if kv_rows.size:
            b_of, p_of = kv_rows // S_act, pos_begin + kv_rows % S_act
            self.k_cache[b_of, p_of] = r16(orc.rope(orc.linear(xn[kv_rows], self.w_k), positions[kv_rows], H, hd, self.theta))
            self.v_cache[b_of, p_of] = r16(orc.linear(xn[kv_rows], self.w_v))
        if not self.has_prev:
            self.kv_len, self.batch = S_act, B
        q_rot = r16(orc.rope(q, positions, H, hd, self.theta))
        at_rows = idx if (mode & orc.MODE_O) else np.arange(T)
        for b in range(B):
            rows_b = at_rows[(at_rows >= b * S_act) & (at_rows < (b + 1) * S_act)]
            if rows_b.size:
                o = orc.attention_rows(q_rot[rows_b], self.k_cache[b, :self.kv_len], self.v_cache[b, :self.kv_len], H, hd)
                self.o_cache[b, pos_begin + rows_b - b * S_act] = r16(o)
        y = orc.linear(self.o_cache[:B, win].reshape(T, d), self.w_o)
        dl = self.delta[:B, win].reshape(T)
        self.delta[:B, win] = np.where(sel, 0, dl + 1).reshape(B, S_act)
        self.has_prev = True
        self.last_scores, self.last_idx = scores, idx.astype(np.int32)
        self.last_batch_off = np.searchsorted(idx, np.arange(B + 1) * S_act).astype(np.int32)
        return y.reshape(B, S_act, d)


def rounded_layer(shape, w, score_head=0):
    return RoundedLayer(shape.d_model, shape.n_heads, shape.head_dim, shape.batch, shape.seq, shape.rope_theta,
                        shape.rms_eps, w["w_q"], w["w_k"], w["w_v"], w["w_o"], w["rms_gain"], score_head=score_head)


def clear_thresholds(score_sets, min_gap=2e-3, limit=8, max_gap=6e-3):
    """Thresholds at the midpoints of gaps that no score of any of the given sets falls into: each token forbids the
    interval between its smallest and its largest score over the sets.  Gaps between `min_gap` and `max_gap` wide come
    first (a threshold there has scores within max_gap / 2 on both sides); wider ones fill up to three thresholds if
    there are too few.  At most `limit`, spread over the range, ascending."""
    s = np.stack([np.asarray(a, np.float64) for a in score_sets])
    lo, hi = s.min(axis=0), s.max(axis=0)
    order = np.argsort(lo)
    lo, hi = lo[order], hi[order]
    reach = np.maximum.accumulate(hi)                 # right end of everything that starts at or before token i
    gaps = [(lo[i + 1] - reach[i], 0.5 * (reach[i] + lo[i + 1])) for i in range(len(lo) - 1) if lo[i + 1] - reach[i] >= min_gap]
    taus = sorted(t for g, t in gaps if g <= max_gap)
    if len(taus) > limit:
        pick = np.unique(np.round(np.linspace(0, len(taus) - 1, limit)).astype(int))
        taus = [taus[i] for i in pick]
    if len(taus) < 3:
        wide = sorted(gaps)                           # narrowest of the wide ones first
        taus = sorted(taus + [t for g, t in wide if g > max_gap][:3 - len(taus)])
    return taus
