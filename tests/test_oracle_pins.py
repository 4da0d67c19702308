"""Pins for the fp64 oracle: every function is checked against something other than itself.

 * library routines in the special cases where the step reduces to one
   (torch rms_norm / linear / cosine_similarity / scaled_dot_product_attention, all fp64 on CPU);
 * closed forms (identical / opposite / orthogonal vectors, uniform softmax, rotations);
 * a pure-Python scalar brute force of the whole layer step on tiny inputs, written with complex
   arithmetic for the rotary embedding and explicit loops everywhere else;
 * invariants the paper states: tau = 0 gives no reuse on perturbed inputs and zero staleness (Sec. 4),
   no reuse in a step means the dense result (Prop. 1), reused rows are the cached rows (Eq. 3, Eq. 4),
   the appendix form of the reuse predicate, the staleness recurrence, the bound of Eq. (x_diff).
"""
import cmath
import math

import numpy as np
import pytest
import torch

from oracle import dare_oracle as orc
from paper_2605_08134_b200 import workloads as wl

RNG = np.random.default_rng(1234)


# ----------------------------------------------------------------------------- library pins
def test_rmsnorm_matches_torch():
    x = RNG.standard_normal((7, 24))
    g = RNG.standard_normal(24)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (24,), torch.from_numpy(g), 1e-5).numpy()
    np.testing.assert_allclose(orc.rmsnorm(x, g, 1e-5), ref, rtol=1e-13, atol=1e-13)


def test_rmsnorm_closed_form():
    # a row of constants c normalises to c/sqrt(c^2+eps) * gain
    x = np.full((1, 16), 3.0)
    out = orc.rmsnorm(x, np.full(16, 2.0), 0.25)
    np.testing.assert_allclose(out, np.full((1, 16), 2.0 * 3.0 / math.sqrt(9.25)), rtol=1e-15)
    # eps = 0, unit gain: every row has norm sqrt(d)
    y = orc.rmsnorm(RNG.standard_normal((5, 32)), np.ones(32), 0.0)
    np.testing.assert_allclose(np.linalg.norm(y, axis=1), math.sqrt(32), rtol=1e-14)


def test_linear_is_w_times_x():
    x = RNG.standard_normal((3, 5))
    w = RNG.standard_normal((4, 5))          # [out, in]
    y = orc.linear(x, w)
    assert y.shape == (3, 4)
    for i in range(3):
        for o in range(4):
            assert abs(y[i, o] - sum(w[o, j] * x[i, j] for j in range(5))) < 1e-13
    ref = torch.nn.functional.linear(torch.from_numpy(x), torch.from_numpy(w)).numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-13, atol=1e-13)


def test_drift_score_closed_forms():
    a = RNG.standard_normal((1, 16))
    assert abs(orc.drift_score(a, a)[0]) < 1e-15                    # identical -> 0
    assert abs(orc.drift_score(a, -a)[0] - 2.0) < 1e-15             # opposite -> 2
    e0, e1 = np.eye(16)[[0]], np.eye(16)[[1]]
    assert orc.drift_score(e0, e1)[0] == 1.0                        # orthogonal -> 1
    b = RNG.standard_normal((1, 16))
    s = orc.drift_score(a, b)[0]
    assert abs(orc.drift_score(3.7 * a, b)[0] - s) < 1e-14          # scale invariant in either argument
    assert abs(orc.drift_score(a, 0.01 * b)[0] - s) < 1e-14
    assert abs(orc.drift_score(b, a)[0] - s) < 1e-15                # symmetric
    # 45 degrees: 1 - cos(pi/4)
    u = np.array([[1.0, 0.0]])
    v = np.array([[1.0, 1.0]])
    assert abs(orc.drift_score(u, v)[0] - (1 - math.sqrt(0.5))) < 1e-15
    # zero vector: cosine taken as 0
    assert orc.drift_score(np.zeros((1, 4)), np.ones((1, 4)))[0] == 1.0


def test_drift_score_matches_torch_cosine():
    a, b = RNG.standard_normal((9, 64)), RNG.standard_normal((9, 64))
    ref = 1 - torch.nn.functional.cosine_similarity(torch.from_numpy(a), torch.from_numpy(b), dim=-1).numpy()
    np.testing.assert_allclose(orc.drift_score(a, b), ref, rtol=1e-12, atol=1e-14)


def test_attention_matches_torch_sdpa():
    S, H, hd, m = 11, 3, 8, 4
    q, k, v = (RNG.standard_normal((n, H * hd)) for n in (m, S, S))
    out = orc.attention_rows(q, k, v, H, hd)
    tq = torch.from_numpy(q).reshape(1, m, H, hd).transpose(1, 2)
    tk = torch.from_numpy(k).reshape(1, S, H, hd).transpose(1, 2)
    tv = torch.from_numpy(v).reshape(1, S, H, hd).transpose(1, 2)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=False)
    ref = ref.transpose(1, 2).reshape(m, H * hd).numpy()
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-13)


def test_attention_closed_forms():
    S, H, hd = 6, 2, 4
    k, v = RNG.standard_normal((S, H * hd)), RNG.standard_normal((S, H * hd))
    # zero query -> uniform weights -> mean of V (weights sum to 1)
    out = orc.attention_rows(np.zeros((1, H * hd)), k, v, H, hd)
    np.testing.assert_allclose(out[0], v.mean(axis=0), rtol=1e-14)
    # one key only -> its value, whatever the query
    out = orc.attention_rows(RNG.standard_normal((2, H * hd)), k[:1], v[:1], H, hd)
    np.testing.assert_allclose(out, np.repeat(v[:1], 2, axis=0), rtol=1e-15)
    # bidirectional: permuting the keys (with their values) leaves the output unchanged
    q = RNG.standard_normal((3, H * hd))
    perm = RNG.permutation(S)
    np.testing.assert_allclose(orc.attention_rows(q, k, v, H, hd),
                               orc.attention_rows(q, k[perm], v[perm], H, hd), rtol=1e-12, atol=1e-14)
    # heads are independent: changing head 1 of K leaves head 0 of the output alone
    k2 = k.copy()
    k2[:, hd:] = RNG.standard_normal((S, hd))
    a, b = orc.attention_rows(q, k, v, H, hd), orc.attention_rows(q, k2, v, H, hd)
    assert np.array_equal(a[:, :hd], b[:, :hd]) and not np.allclose(a[:, hd:], b[:, hd:])
    # a huge logit picks out one key: scale is 1/sqrt(head_dim), sign positive
    qq = np.zeros((1, H * hd)); qq[0, 0] = 1e4; qq[0, hd] = 1e4
    kk = np.zeros((S, H * hd)); kk[2, 0] = 1.0; kk[4, hd] = 1.0
    out = orc.attention_rows(qq, kk, v, H, hd)
    np.testing.assert_allclose(out[0, :hd], v[2, :hd], rtol=1e-12)
    np.testing.assert_allclose(out[0, hd:], v[4, hd:], rtol=1e-12)


def test_attention_scale_is_inv_sqrt_head_dim():
    # two keys, one head: weights are softmax([q.k0, q.k1]/sqrt(hd)) exactly
    hd = 16
    q = np.zeros((1, hd)); q[0, 0] = 2.0
    k = np.zeros((2, hd)); k[0, 0] = 3.0; k[1, 0] = -1.0
    v = np.zeros((2, hd)); v[0, 1] = 1.0; v[1, 2] = 1.0
    out = orc.attention_rows(q, k, v, 1, hd)
    l0, l1 = 6.0 / 4.0, -2.0 / 4.0
    p0 = math.exp(l0) / (math.exp(l0) + math.exp(l1))
    assert abs(out[0, 1] - p0) < 1e-15 and abs(out[0, 2] - (1 - p0)) < 1e-15


# ----------------------------------------------------------------------------- rotary embedding
def test_rope_properties():
    H, hd, theta = 2, 8, 1e4
    v = RNG.standard_normal((5, H * hd))
    pos = np.array([0, 1, 2, 7, 100])
    r = orc.rope(v, pos, H, hd, theta)
    np.testing.assert_array_equal(r[0], v[0])                                   # position 0: identity
    vh, rh = v.reshape(5, H, hd), r.reshape(5, H, hd)
    np.testing.assert_allclose(np.linalg.norm(rh, axis=-1), np.linalg.norm(vh, axis=-1), rtol=1e-13)
    # complex form: (a_j + i b_j) * exp(i * pos * theta^(-2j/hd)) with b_j = element j + hd/2
    for row in range(5):
        for h in range(H):
            for j in range(hd // 2):
                z = complex(vh[row, h, j], vh[row, h, j + hd // 2]) * cmath.exp(1j * pos[row] * theta ** (-2 * j / hd))
                assert abs(z.real - rh[row, h, j]) < 1e-12 and abs(z.imag - rh[row, h, j + hd // 2]) < 1e-12
    # relative-position property: <R_m q, R_n k> depends on m - n only
    q, k = RNG.standard_normal((1, hd)), RNG.standard_normal((1, hd))
    d1 = orc.rope(q, [5], 1, hd, theta) @ orc.rope(k, [3], 1, hd, theta).T
    d2 = orc.rope(q, [42], 1, hd, theta) @ orc.rope(k, [40], 1, hd, theta).T
    assert abs(d1 - d2) < 1e-12
    # the slowest pair turns by pos * theta^(-(hd-2)/hd)
    e = np.zeros((1, hd)); e[0, hd // 2 - 1] = 1.0
    out = orc.rope(e, [10], 1, hd, theta)
    ang = 10 * theta ** (-(hd - 2) / hd)
    assert abs(out[0, hd // 2 - 1] - math.cos(ang)) < 1e-14 and abs(out[0, hd - 1] - math.sin(ang)) < 1e-14


def test_score_is_rotation_invariant():
    """Scoring before or after the rotary embedding gives the same number (same position for both vectors)."""
    hd = 64
    a, b = RNG.standard_normal((6, hd)), RNG.standard_normal((6, hd))
    pos = np.array([0, 3, 17, 64, 255, 511])
    s_plain = orc.drift_score(a, b)
    s_rot = orc.drift_score(orc.rope(a, pos, 1, hd, 5e5), orc.rope(b, pos, 1, hd, 5e5))
    np.testing.assert_allclose(s_plain, s_rot, rtol=0, atol=1e-12)


# ----------------------------------------------------------------------------- selection
def test_refresh_mask_predicate():
    s = np.array([0.0, 0.05, 0.1, 0.1000001, 0.5, np.nan, np.inf])
    np.testing.assert_array_equal(orc.refresh_mask(s, 0.1), [False, False, False, True, True, True, True])
    assert orc.refresh_mask(s, -1.0).all()                          # tau < 0: everything refreshed
    np.testing.assert_array_equal(orc.refresh_mask(s, np.inf), [False] * 5 + [True, False])   # NaN stays refreshed
    # tau = 0 with an exactly-zero score: Eq. 2 has "<=", so that token is reused
    assert not orc.refresh_mask(np.array([0.0]), 0.0)[0]


def test_appendix_form_of_predicate():
    """Appendix E: R = {i : <q_hat_t, q_hat_{t-1}> >= 1 - tau} on unit-normalised queries is the same set."""
    a, b = RNG.standard_normal((200, 16)), RNG.standard_normal((200, 16))
    b[:100] = a[:100] + 0.2 * b[:100]
    an, bn = a / np.linalg.norm(a, axis=1, keepdims=True), b / np.linalg.norm(b, axis=1, keepdims=True)
    for tau in (0.01, 0.05, 0.3, 1.0):
        reuse_appendix = np.sum(an * bn, axis=1) >= 1 - tau
        np.testing.assert_array_equal(~orc.refresh_mask(orc.drift_score(a, b), tau), reuse_appendix)


# ----------------------------------------------------------------------------- brute force of the whole step
class BruteLayer:
    """Scalar, loop-only restatement of Alg. 1 / Alg. 2 / both for one sequence batch (tiny sizes)."""

    def __init__(self, d, H, hd, theta, eps, wq, wk, wv, wo, gain, score_head=0):
        self.d, self.H, self.hd, self.theta, self.eps = d, H, hd, theta, eps
        self.score_head = score_head
        self.wq, self.wk, self.wv, self.wo, self.gain = (np.asarray(a, float).tolist() for a in (wq, wk, wv, wo, gain))
        self.prev = None

    def _matvec(self, w, x):
        return [sum(w[o][j] * x[j] for j in range(self.d)) for o in range(self.d)]

    def _rot(self, vec, pos):
        out = list(vec)
        half = self.hd // 2
        for h in range(self.H):
            for j in range(half):
                z = complex(vec[h * self.hd + j], vec[h * self.hd + j + half])
                z *= cmath.exp(1j * pos * self.theta ** (-2.0 * j / self.hd))
                out[h * self.hd + j], out[h * self.hd + j + half] = z.real, z.imag
        return out

    def step(self, x, mode, tau):
        B, S, d = len(x), len(x[0]), self.d
        H, hd = self.H, self.hd
        first = self.prev is None
        if first:
            self.qp = [[None] * S for _ in range(B)]
            self.K = [[None] * S for _ in range(B)]
            self.V = [[None] * S for _ in range(B)]
            self.O = [[None] * S for _ in range(B)]
            self.delta = [[0] * S for _ in range(B)]
        xn = [[None] * S for _ in range(B)]
        q = [[None] * S for _ in range(B)]
        sel = [[True] * S for _ in range(B)]
        scores = [[math.inf] * S for _ in range(B)]
        for b in range(B):
            for i in range(S):
                ms = sum(t * t for t in x[b][i]) / d
                xn[b][i] = [x[b][i][j] / math.sqrt(ms + self.eps) * self.gain[j] for j in range(d)]
                q[b][i] = self._matvec(self.wq, xn[b][i])
                q0 = q[b][i][self.score_head * hd:(self.score_head + 1) * hd]
                if not first:
                    p = self.qp[b][i]
                    dot = sum(u * w for u, w in zip(q0, p))
                    na, nb = math.sqrt(sum(u * u for u in q0)), math.sqrt(sum(u * u for u in p))
                    scores[b][i] = 1.0 - dot / (na * nb)
                    if mode != 0:
                        sel[b][i] = not (scores[b][i] <= tau)
                self.qp[b][i] = q0
        for b in range(B):
            for i in range(S):
                if sel[b][i] or not (mode & 1):
                    self.K[b][i] = self._rot(self._matvec(self.wk, xn[b][i]), i)
                    self.V[b][i] = self._matvec(self.wv, xn[b][i])
        for b in range(B):
            for i in range(S):
                if not (sel[b][i] or not (mode & 2)):
                    continue
                qr = self._rot(q[b][i], i)
                o = [0.0] * d
                for h in range(H):
                    lo = h * hd
                    logit = [sum(qr[lo + c] * self.K[b][j][lo + c] for c in range(hd)) / math.sqrt(hd) for j in range(S)]
                    mx = max(logit)
                    w = [math.exp(l - mx) for l in logit]
                    z = sum(w)
                    for c in range(hd):
                        o[lo + c] = sum(w[j] / z * self.V[b][j][lo + c] for j in range(S))
                self.O[b][i] = o
        y = [[self._matvec(self.wo, self.O[b][i]) for i in range(S)] for b in range(B)]
        for b in range(B):
            for i in range(S):
                self.delta[b][i] = 0 if sel[b][i] else self.delta[b][i] + 1
        self.prev = True
        return np.array(y), np.array(scores), np.array(sel)


def _tiny(seed, B=2, S=5, d=8, H=2):
    rng = np.random.default_rng(seed)
    hd = d // H
    ws = [rng.standard_normal((d, d)) * 0.3 for _ in range(4)]
    gain = 1.0 + 0.1 * rng.standard_normal(d)
    xs = [rng.standard_normal((B, S, d))]
    for _ in range(3):
        nxt = xs[-1] + 1e-3 * rng.standard_normal((B, S, d))
        redo = rng.random((B, S)) < 0.4
        nxt[redo] = rng.standard_normal((int(redo.sum()), d))
        xs.append(nxt)
    return (B, S, d, H, hd), ws, gain, xs


@pytest.mark.parametrize("mode", [orc.MODE_DENSE, orc.MODE_KV, orc.MODE_O, orc.MODE_BOTH])
@pytest.mark.parametrize("seed", [0, 1])
def test_step_matches_brute_force(mode, seed):
    (B, S, d, H, hd), ws, gain, xs = _tiny(seed)
    lay = orc.OracleLayer(d, H, hd, B, S, 100.0, 1e-5, *ws, gain)
    bru = BruteLayer(d, H, hd, 100.0, 1e-5, *ws, gain)
    for t, x in enumerate(xs):
        y = lay.step(x, mode, 0.05)
        yb, sb, selb = bru.step(x.tolist(), mode, 0.05)
        np.testing.assert_allclose(y, yb, rtol=1e-10, atol=1e-12)
        if t > 0:
            np.testing.assert_allclose(lay.last_scores, sb.reshape(-1), rtol=1e-9, atol=1e-13)
        np.testing.assert_array_equal(lay.last_idx, np.nonzero(selb.reshape(-1))[0])
        np.testing.assert_array_equal(lay.delta[:B, :S], np.array(bru.delta))
        np.testing.assert_allclose(lay.k_cache[:B, :S], np.array(bru.K), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(lay.v_cache[:B, :S], np.array(bru.V), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(lay.o_cache[:B, :S], np.array(bru.O), rtol=1e-10, atol=1e-12)
        if t > 0 and mode != 0:
            assert 0 < len(lay.last_idx) < B * S        # the case really mixes reuse and refresh


@pytest.mark.parametrize("mode", [orc.MODE_KV, orc.MODE_BOTH])
def test_step_matches_brute_force_with_another_scoring_head(mode):
    """Sec. 3.2 scores head 0; the head is a parameter of the layer.  With head 1 the scalar restatement and the oracle
    must still agree, and the refresh set must differ from head 0's somewhere (the parameter does something)."""
    (B, S, d, H, hd), ws, gain, xs = _tiny(5, B=2, S=6)
    lay = orc.OracleLayer(d, H, hd, B, S, 100.0, 1e-5, *ws, gain, score_head=1)
    ref0 = orc.OracleLayer(d, H, hd, B, S, 100.0, 1e-5, *ws, gain, score_head=0)
    bru = BruteLayer(d, H, hd, 100.0, 1e-5, *ws, gain, score_head=1)
    differs = False
    for t, x in enumerate(xs):
        y = lay.step(x, mode, 0.05)
        ref0.step(x, mode, 0.05)
        yb, sb, selb = bru.step(x.tolist(), mode, 0.05)
        np.testing.assert_allclose(y, yb, rtol=1e-10, atol=1e-12)
        if t > 0:
            np.testing.assert_allclose(lay.last_scores, sb.reshape(-1), rtol=1e-9, atol=1e-13)
            differs |= not np.allclose(lay.last_scores, ref0.last_scores)
        np.testing.assert_array_equal(lay.last_idx, np.nonzero(selb.reshape(-1))[0])
        np.testing.assert_allclose(lay.q_prev[:B, :S], np.array(bru.qp), rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(lay.o_cache[:B, :S], np.array(bru.O), rtol=1e-10, atol=1e-12)
    assert differs


@pytest.mark.parametrize("score_head", [0, 2])
def test_scores_only_is_the_score_of_the_step(score_head):
    """`scores_only` (lines 1-3 of Alg. 1 without the state update) against what the full step then reports, on full
    and on window steps; it must leave the state alone and report +inf before a first step."""
    shape = wl.scaled(wl.TINY_F32, d_model=64, n_heads=4, head_dim=16, seq=48, prompt=16, batch=2)
    w = wl.make_weights(shape, 17)
    hs = wl.HiddenStream(shape, 17)
    lay = orc.OracleLayer(shape.d_model, shape.n_heads, shape.head_dim, shape.batch, shape.seq, shape.rope_theta,
                          shape.rms_eps, w["w_q"], w["w_k"], w["w_v"], w["w_o"], w["rms_gain"], score_head=score_head)
    x0 = hs.first()
    assert np.isinf(orc.scores_only(lay, x0)).all()
    lay.step(x0, 3, 0.1)
    for t in range(3):
        x = hs.advance_graded() if t == 1 else hs.advance(wl.uniform_positions(hs.rng, shape, 9))
        p = 16 if t == 2 else 0
        xw = np.ascontiguousarray(x[:, p:])
        before = (lay.q_prev.copy(), lay.k_cache.copy(), lay.o_cache.copy(), lay.delta.copy())
        s = orc.scores_only(lay, xw, pos_begin=p)
        for a, b in zip(before, (lay.q_prev, lay.k_cache, lay.o_cache, lay.delta)):
            np.testing.assert_array_equal(a, b)
        lay.step(xw, 3, 0.1, pos_begin=p)
        np.testing.assert_allclose(s, lay.last_scores, rtol=1e-12, atol=1e-15)
        assert 0 < len(lay.last_idx) < xw.shape[0] * xw.shape[1]


# ----------------------------------------------------------------------------- invariants of the method
def _small_case(dtype=wl.DTYPE_F32, changed=6, seed=3, **kw):
    shape = wl.scaled(wl.TINY_F32, d_model=64, n_heads=4, head_dim=16, seq=32, prompt=16, batch=2, dtype=dtype, **kw)
    w, x0, x1, ch = wl.two_step_case(shape, changed, seed)
    return shape, w, x0, x1, ch


def _layer(shape, w):
    return orc.OracleLayer(shape.d_model, shape.n_heads, shape.head_dim, shape.batch, shape.seq,
                           shape.rope_theta, shape.rms_eps, w["w_q"], w["w_k"], w["w_v"], w["w_o"], w["rms_gain"])


def test_first_step_is_dense_and_selects_everything():
    shape, w, x0, _, _ = _small_case()
    outs = []
    for mode in (0, 1, 2, 3):
        lay = _layer(shape, w)
        outs.append(lay.step(x0, mode, 0.1))
        assert len(lay.last_idx) == shape.tokens and np.isinf(lay.last_scores).all()
        assert (lay.delta == 0).all()
    for o in outs[1:]:
        np.testing.assert_array_equal(o, outs[0])


@pytest.mark.parametrize("mode", [1, 2, 3])
def test_no_reuse_equals_dense(mode):
    """Prop. 1 / Sec. 4: a step without reuse has no error.  tau < 0 refreshes all; tau = 0 does on perturbed inputs."""
    shape, w, x0, x1, _ = _small_case()
    dense = _layer(shape, w); dense.step(x0, 0, 0.0); yd = dense.step(x1, 0, 0.0)
    for tau in (-1.0, 0.0):
        lay = _layer(shape, w); lay.step(x0, mode, tau)
        y = lay.step(x1, mode, tau)
        assert lay.last_scores.min() > 0                            # every token was perturbed
        assert len(lay.last_idx) == shape.tokens
        np.testing.assert_array_equal(y, yd)
        assert (lay.delta == 0).all()                               # tau = 0 => delta == 0 (Sec. 4)


@pytest.mark.parametrize("mode", [1, 2, 3])
def test_reuse_everything_at_infinite_threshold(mode):
    shape, w, x0, x1, _ = _small_case()
    lay = _layer(shape, w)
    y0 = lay.step(x0, mode, np.inf)
    k0, v0, o0 = lay.k_cache.copy(), lay.v_cache.copy(), lay.o_cache.copy()
    y1 = lay.step(x1, mode, np.inf)
    assert len(lay.last_idx) == 0
    if mode & 1:
        assert np.array_equal(lay.k_cache, k0) and np.array_equal(lay.v_cache, v0)
    if mode & 2:
        assert np.array_equal(lay.o_cache, o0)
        np.testing.assert_array_equal(y1, y0)                       # all outputs reused -> same projection
    assert (lay.delta[:shape.batch] == 1).all()


def test_selected_set_is_the_changed_set_and_reused_rows_are_bit_identical():
    """Eq. 3 / Eq. 4: rows in the reuse set are literally the cached rows."""
    shape, w, x0, x1, changed = _small_case()
    planned = np.nonzero(changed.reshape(-1))[0]
    for mode in (1, 2, 3):
        lay = _layer(shape, w)
        lay.step(x0, mode, 0.1)
        k0, v0, o0 = lay.k_cache.copy(), lay.v_cache.copy(), lay.o_cache.copy()
        lay.step(x1, mode, 0.1)
        np.testing.assert_array_equal(lay.last_idx, planned)
        keep = ~changed
        if mode & 1:
            assert np.array_equal(lay.k_cache[keep], k0[keep]) and np.array_equal(lay.v_cache[keep], v0[keep])
            assert not np.allclose(lay.k_cache[changed], k0[changed])
        else:
            assert not np.array_equal(lay.k_cache[keep], k0[keep])   # dense K/V moved (tiny noise)
        if mode & 2:
            assert np.array_equal(lay.o_cache[keep], o0[keep])
        assert not np.allclose(lay.o_cache[changed], o0[changed])


def test_one_changed_token_changes_one_cache_row():
    shape, w, x0, _, _ = _small_case()
    x1 = x0.copy()
    x1[1, 7] = np.random.default_rng(5).standard_normal(shape.d_model).astype(np.float32)
    lay = _layer(shape, w)
    lay.step(x0, orc.MODE_KV, 1e-9)
    k0 = lay.k_cache.copy()
    lay.step(x1, orc.MODE_KV, 1e-9)       # unchanged rows score 0 up to rounding (~1e-16): reused
    np.testing.assert_array_equal(lay.last_idx, [1 * shape.seq + 7])
    diff = np.any(lay.k_cache != k0, axis=-1)
    assert diff.sum() == 1 and diff[1, 7]


def test_selected_o_rows_equal_dense_attention_over_current_cache():
    shape, w, x0, x1, changed = _small_case()
    lay = _layer(shape, w)
    lay.step(x0, 3, 0.1)
    lay.step(x1, 3, 0.1)
    T = shape.tokens
    xn = orc.rmsnorm(np.asarray(x1, float).reshape(T, -1), w["rms_gain"], shape.rms_eps)
    pos = np.tile(np.arange(shape.seq), shape.batch)
    q = orc.rope(orc.linear(xn, w["w_q"]), pos, shape.n_heads, shape.head_dim, shape.rope_theta)
    for b in range(shape.batch):
        full = orc.attention_rows(q[b * shape.seq:(b + 1) * shape.seq], lay.k_cache[b], lay.v_cache[b],
                                  shape.n_heads, shape.head_dim)
        np.testing.assert_allclose(lay.o_cache[b][changed[b]], full[changed[b]], rtol=1e-12, atol=1e-14)


def test_both_is_kv_then_o_composed_by_hand():
    shape, w, x0, x1, changed = _small_case()
    both = _layer(shape, w); both.step(x0, 3, 0.1); y_both = both.step(x1, 3, 0.1)
    kv = _layer(shape, w); kv.step(x0, 1, 0.1)
    o_prev = kv.o_cache.copy()
    kv.step(x1, 1, 0.1)                    # hybrid cache + attention on every row
    o_hand = np.where(changed[:, :, None], kv.o_cache, o_prev)
    np.testing.assert_array_equal(both.k_cache, kv.k_cache)
    np.testing.assert_allclose(both.o_cache, o_hand, rtol=1e-13, atol=1e-15)
    y_hand = orc.linear(o_hand.reshape(shape.tokens, -1), w["w_o"]).reshape(y_both.shape)
    np.testing.assert_allclose(y_both, y_hand, rtol=1e-13, atol=1e-15)


def test_output_projection_commutes_with_row_reuse():
    """W_O acts row-wise, so caching the projected rows and projecting only refreshed rows gives the same output."""
    shape, w, x0, x1, changed = _small_case()
    lay = _layer(shape, w)
    y0 = lay.step(x0, 2, 0.1)
    y1 = lay.step(x1, 2, 0.1)
    keep = ~changed
    np.testing.assert_allclose(y1[keep], y0[keep], rtol=0, atol=1e-12)
    assert not np.allclose(y1[changed], y0[changed])


def test_selection_is_monotone_and_nested_in_threshold():
    shape = wl.scaled(wl.TINY_F32, d_model=64, n_heads=4, head_dim=16, seq=64, prompt=32, batch=2)
    w = wl.make_weights(shape, 11)
    hs = wl.HiddenStream(shape, 11)
    x0 = hs.first()
    x1 = hs.advance_graded()
    probe = _layer(shape, w); probe.step(x0, 0, 0.0)
    s = np.sort(orc.scores_only(probe, x1))
    assert s[0] < 1e-4 and s[-1] > 0.1                              # scores spread over decades
    gaps = np.nonzero(np.diff(s) >= 2e-3)[0]
    taus = [-1.0] + [0.5 * (s[g] + s[g + 1]) for g in gaps] + [np.inf]
    assert len(taus) >= 4
    prev = None
    for tau in taus:
        lay = _layer(shape, w); lay.step(x0, 3, tau); lay.step(x1, 3, tau)
        cur = set(lay.last_idx.tolist())
        if prev is not None:
            assert cur <= prev                                      # larger tau refreshes a subset
        prev = cur
    assert len(prev) == 0


def test_staleness_recurrence_over_many_steps():
    shape = wl.scaled(wl.TINY_F32, d_model=64, n_heads=4, head_dim=16, seq=32, prompt=16, batch=2)
    w = wl.make_weights(shape, 2)
    hs = wl.HiddenStream(shape, 2)
    lay = _layer(shape, w)
    lay.step(hs.first(), 3, 0.1)
    expect = np.zeros((shape.batch, shape.seq), int)
    for t in range(6):
        ch = wl.uniform_positions(hs.rng, shape, 5)
        lay.step(hs.advance(ch), 3, 0.1)
        np.testing.assert_array_equal(lay.last_idx, np.nonzero(ch.reshape(-1))[0])
        expect = np.where(ch, 0, expect + 1)
        np.testing.assert_array_equal(lay.delta, expect)
    assert expect.max() == 6 or expect.max() >= 3


def test_batch_offsets_and_independent_sequences():
    shape, w, x0, x1, changed = _small_case()
    lay = _layer(shape, w); lay.step(x0, 3, 0.1); y = lay.step(x1, 3, 0.1)
    off = lay.last_batch_off
    assert off[0] == 0 and off[-1] == len(lay.last_idx)
    for b in range(shape.batch):
        assert off[b + 1] - off[b] == changed[b].sum()
    # running sequence 1 alone gives the same rows
    s1 = wl.scaled(shape, batch=1)
    solo = _layer(s1, w); solo.step(x0[1:2], 3, 0.1); ys = solo.step(x1[1:2], 3, 0.1)
    np.testing.assert_allclose(y[1], ys[0], rtol=1e-12, atol=1e-14)


def test_window_step_keeps_prefix_rows():
    """A step over positions [p, p+n) scores and refreshes only those rows; the others keep their caches."""
    shape, w, x0, x1, _ = _small_case()
    p = 16
    lay = _layer(shape, w)
    lay.step(x0, 3, 0.1)
    k0, o0 = lay.k_cache.copy(), lay.o_cache.copy()
    y = lay.step(x1[:, p:], 0, 0.0, pos_begin=p)                    # dense over the window
    assert np.array_equal(lay.k_cache[:, :p], k0[:, :p]) and np.array_equal(lay.o_cache[:, :p], o0[:, :p])
    assert not np.allclose(lay.k_cache[:, p:], k0[:, p:])
    # window rows attend over the frozen prefix + fresh window: rebuild by hand
    full = _layer(shape, w)
    full.step(x0, 0, 0.0)
    mixed = np.concatenate([x0[:, :p], x1[:, p:]], axis=1)
    yf = full.step(mixed, 0, 0.0)
    np.testing.assert_allclose(y, yf[:, p:], rtol=1e-12, atol=1e-14)


def test_x_diff_bound_for_reused_tokens():
    """Eq. (x_diff): for a reused token, |x_hat_t - x_hat_{t-1}|^2 <= 4 d tau kappa^2 / (2 + tau (kappa^2 - 1)),
    single head scoring the full query, unit-gain normalisation with eps = 0 (so |x_hat| = sqrt(d))."""
    d = 16
    rng = np.random.default_rng(9)
    u, _ = np.linalg.qr(rng.standard_normal((d, d)))
    v, _ = np.linalg.qr(rng.standard_normal((d, d)))
    sv = np.linspace(1.0, 3.0, d)
    wq = u @ np.diag(sv) @ v.T
    kappa = 3.0
    x0 = rng.standard_normal((400, d))
    x1 = x0 + rng.uniform(0, 0.6, (400, 1)) * rng.standard_normal((400, d))
    xn0, xn1 = orc.rmsnorm(x0, np.ones(d), 0.0), orc.rmsnorm(x1, np.ones(d), 0.0)
    s = orc.drift_score(orc.linear(xn1, wq), orc.linear(xn0, wq))
    for tau in (0.01, 0.05, 0.2):
        reused = ~orc.refresh_mask(s, tau)
        assert reused.any() and (~reused).any()
        bound = 4 * d * tau * kappa ** 2 / (2 + tau * (kappa ** 2 - 1))
        lhs = np.sum((xn1 - xn0) ** 2, axis=1)
        assert (lhs[reused] <= bound + 1e-12).all()


def test_nan_threshold_rejected_and_shapes_checked():
    shape, w, x0, _, _ = _small_case()
    lay = _layer(shape, w)
    with pytest.raises(ValueError):
        lay.step(x0, 1, float("nan"))
