"""fp64 CPU oracle for DARE's per-layer activation-reuse attention step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
CUDA library must compute.  It shares no code with the CUDA path and must never
be imported by the product package; only the test-suite, the smoke check and
the CPU-baseline leg of the benchmark call it.

Everything is numpy float64.  The method is an approximation with state (it is
not a faster route to the dense result), so the oracle is the algorithm itself,
taken step by step in the paper's order:

  Algorithm 1 (DARE-KV), Algorithm 2 (DARE-O), Sec. 3.1 (drift score),
  Eq. 2 (reuse set), Eq. 3 (K/V refresh), Eq. 4 (output reuse),
  Sec. 4 (staleness counter).

A numpy matmul serves as the "linear layer" primitive; nothing is blocked,
fused or reordered beyond what the algorithms state.

Readings taken where the paper is silent (each one is listed with its reason in
the design notes of the repository):
  * first step after creation/reset: no previous query exists, every token is
    refreshed (score = +inf);
  * "LayerNorm" of Alg. 1/2 line 1 is RMSNorm with a gain vector (LLaDA layer);
  * rotary embedding, half-split pairing (element j with j + head_dim/2), is
    applied to Q for attention and to K before it is cached; the drift score is
    taken on the un-rotated head-0 query (a rotation common to both vectors
    does not change a cosine);
  * softmax scale 1/sqrt(head_dim) (the appendix's 1/sqrt(d) for one head);
  * weights use the W[out, in] convention, y = W x (Alg. 1 line 2);
  * zero-norm query: cosine := 0, score = 1;  NaN score: token refreshed,
    because the refresh set is the complement of {s <= tau} (Alg. 1 line 5);
  * "both": Eq. 3 and Eq. 4 driven by the one index set of the step;
  * batch > 1: one flat ascending index list over the active tokens, attention
    never crosses sequences.

Parity pins: every function below is pinned by tests/test_oracle_*.py (closed
forms, library routines in special cases, brute force on tiny inputs,
invariants of Sec. 4).  Nothing about model accuracy on real text is pinned
("parity unpinned" for that: it needs trained weights and benchmark suites).
"""
from __future__ import annotations

import numpy as np

MODE_DENSE = 0
MODE_KV = 1      # bit 0: reuse cached K/V for tokens in the reuse set
MODE_O = 2       # bit 1: reuse cached attention outputs for tokens in the reuse set
MODE_BOTH = 3

_F = np.float64


def rmsnorm(x, gain, eps):
    """Alg. 1/2 line 1 (read as RMSNorm): x / sqrt(mean(x^2) + eps) * gain, per token row."""
    x = np.asarray(x, _F)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * np.asarray(gain, _F)


def linear(x, w):
    """Alg. 1 line 2 / line 7: y_i = W x_i with W stored [out, in]."""
    return np.asarray(x, _F) @ np.asarray(w, _F).T


def rope(v, positions, n_heads, head_dim, theta):
    """Rotary position embedding, half-split pairing.

    v: [rows, n_heads*head_dim]; positions: [rows] integer position of each row in
    its sequence.  Within each head, the pair (j, j + head_dim/2) is rotated by the
    angle pos * theta**(-2j/head_dim), j in [0, head_dim/2).
    """
    v = np.asarray(v, _F)
    rows = v.shape[0]
    half = head_dim // 2
    j = np.arange(half, dtype=_F)
    inv_freq = theta ** (-2.0 * j / head_dim)
    ang = np.asarray(positions, _F)[:, None] * inv_freq[None, :]          # [rows, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    vh = v.reshape(rows, n_heads, head_dim)
    a, b = vh[:, :, :half], vh[:, :, half:]
    out = np.empty_like(vh)
    out[:, :, :half] = a * c - b * s
    out[:, :, half:] = a * s + b * c
    return out.reshape(rows, n_heads * head_dim)


def drift_score(q_now, q_prev):
    """Sec. 3.1 drift score per row: s = 1 - <a, b> / (|a| |b|).

    Rows whose either norm is zero get cosine 0 (score 1).
    """
    a = np.asarray(q_now, _F)
    b = np.asarray(q_prev, _F)
    dot = np.sum(a * b, axis=-1)
    na = np.sqrt(np.sum(a * a, axis=-1))
    nb = np.sqrt(np.sum(b * b, axis=-1))
    den = na * nb
    cos = np.zeros_like(dot)
    ok = den > 0
    cos[ok] = dot[ok] / den[ok]
    return 1.0 - cos


def refresh_mask(scores, tau):
    """Eq. 2 and its complement: reuse set R = {i : s_i <= tau}; refreshed = not in R.

    Written as the complement so that a NaN score lands in the refresh set.
    """
    scores = np.asarray(scores, _F)
    with np.errstate(invalid="ignore"):
        reuse = scores <= tau
    return ~reuse


def attention_rows(q_rows, k, v, n_heads, head_dim):
    """Bidirectional softmax attention for the given query rows over all keys.

    q_rows: [m, d], k, v: [S, d] (one sequence).  Per head h:
      O[i, h] = sum_j softmax_j(<q[i,h], k[j,h]> / sqrt(head_dim)) v[j, h],  no mask.
    """
    q_rows = np.asarray(q_rows, _F)
    k = np.asarray(k, _F)
    v = np.asarray(v, _F)
    m = q_rows.shape[0]
    out = np.empty((m, n_heads * head_dim), _F)
    scale = 1.0 / np.sqrt(_F(head_dim))
    for h in range(n_heads):
        sl = slice(h * head_dim, (h + 1) * head_dim)
        logits = (q_rows[:, sl] @ k[:, sl].T) * scale                   # [m, S]
        logits = logits - np.max(logits, axis=1, keepdims=True)
        p = np.exp(logits)
        p = p / np.sum(p, axis=1, keepdims=True)
        out[:, sl] = p @ v[:, sl]
    return out


class OracleLayer:
    """State and step of one DARE attention layer (Alg. 1, Alg. 2 and their union).

    State: previous head-`score_head` query of every token (Sec. 3.2: the stored query
    of the previous diffusion step), the K/V cache (post-rotation K), the cache of
    attention outputs taken before W_O (Alg. 2 lines 9-11), the staleness counter
    (Sec. 4) and `kv_len`, the extent of each sequence that the caches cover.
    """

    def __init__(self, d_model, n_heads, head_dim, max_batch, max_seq, rope_theta, rms_eps,
                 w_q, w_k, w_v, w_o, rms_gain, score_head=0):
        assert n_heads * head_dim == d_model
        self.d, self.H, self.hd = d_model, n_heads, head_dim
        self.max_batch, self.max_seq = max_batch, max_seq
        self.theta, self.eps = float(rope_theta), float(rms_eps)
        self.score_head = score_head
        self.w_q = np.asarray(w_q, _F)
        self.w_k = np.asarray(w_k, _F)
        self.w_v = np.asarray(w_v, _F)
        self.w_o = np.asarray(w_o, _F)
        self.gain = np.asarray(rms_gain, _F)
        self.reset()

    def reset(self):
        B, S, d, hd = self.max_batch, self.max_seq, self.d, self.hd
        self.has_prev = False
        self.batch = 0
        self.kv_len = 0
        self.q_prev = np.zeros((B, S, hd), _F)
        self.k_cache = np.zeros((B, S, d), _F)
        self.v_cache = np.zeros((B, S, d), _F)
        self.o_cache = np.zeros((B, S, d), _F)
        self.delta = np.zeros((B, S), np.int64)
        self.last_scores = None
        self.last_idx = None
        self.last_batch_off = None

    def step(self, x, mode, tau, pos_begin=0, adopt=None):
        """One denoising step.  x: [batch, seq_act, d] covering positions
        [pos_begin, pos_begin + seq_act) of every sequence.  Returns y of the same shape.

        Side outputs kept on the object: last_scores [batch*seq_act], last_idx (ascending
        flat indices b*seq_act + i of refreshed tokens), last_batch_off [batch+1].

        adopt = (other_mask [batch*seq_act] bool, margin): for comparisons with another implementation inside a
        long trajectory.  A token whose score lies within `margin` of tau has no well-defined side; there, and only
        there, the other implementation's decision is taken, so that both keep walking the same trajectory.
        """
        x = np.asarray(x, _F)
        B, S_act, d = x.shape
        H, hd = self.H, self.hd
        assert d == self.d and B <= self.max_batch and pos_begin + S_act <= self.max_seq
        if np.isnan(tau):
            raise ValueError("threshold is NaN")
        if self.has_prev:
            assert B == self.batch and pos_begin + S_act <= self.kv_len
        else:
            assert pos_begin == 0
        win = slice(pos_begin, pos_begin + S_act)
        T = B * S_act
        positions = np.tile(np.arange(pos_begin, pos_begin + S_act), B)

        # Alg. 1/2 line 1: normalise.  line 2: dense query projection for every token.
        xn = rmsnorm(x.reshape(T, d), self.gain, self.eps)
        q = linear(xn, self.w_q)
        sh = self.score_head
        q0 = q[:, sh * hd:(sh + 1) * hd]

        # line 3: drift score of the scoring head against the previous step's query.
        if self.has_prev:
            scores = drift_score(q0, self.q_prev[:B, win].reshape(T, hd))
        else:
            scores = np.full(T, np.inf, _F)
        # lines 4-5: reuse set and its complement.
        if mode == MODE_DENSE or not self.has_prev:
            sel = np.ones(T, bool)          # nothing to compare with, or dense recompute asked for
        else:
            sel = refresh_mask(scores, tau)
            if adopt is not None and self.has_prev:
                other, margin = adopt
                near = np.abs(scores - tau) < margin
                sel = np.where(near, np.asarray(other, bool), sel)
        idx = np.nonzero(sel)[0]

        # Sec. 3.2: the stored query is that of the immediately previous step, for every token.
        self.q_prev[:B, win] = q0.reshape(B, S_act, hd)

        # K/V: Alg. 1 lines 6-9 (refresh selected rows only) or Alg. 2 line 7 (all rows).
        kv_rows = idx if (mode & MODE_KV) else np.arange(T)
        if kv_rows.size:
            k_new = rope(linear(xn[kv_rows], self.w_k), positions[kv_rows], H, hd, self.theta)
            v_new = linear(xn[kv_rows], self.w_v)
            b_of, p_of = kv_rows // S_act, pos_begin + kv_rows % S_act
            self.k_cache[b_of, p_of] = k_new
            self.v_cache[b_of, p_of] = v_new
        if not self.has_prev:
            self.kv_len = S_act
            self.batch = B

        # Attention: Alg. 1 line 10 (all query rows) or Alg. 2 lines 6, 8-10 / Eq. 4 (selected rows).
        q_rot = rope(q, positions, H, hd, self.theta)
        at_rows = idx if (mode & MODE_O) else np.arange(T)
        for b in range(B):
            rows_b = at_rows[(at_rows >= b * S_act) & (at_rows < (b + 1) * S_act)]
            if rows_b.size == 0:
                continue
            o = attention_rows(q_rot[rows_b], self.k_cache[b, :self.kv_len],
                               self.v_cache[b, :self.kv_len], H, hd)
            self.o_cache[b, pos_begin + rows_b - b * S_act] = o

        # Alg. 1 line 11 / Alg. 2 line 11: output projection on every row.
        y = linear(self.o_cache[:B, win].reshape(T, d), self.w_o)

        # Sec. 4: consecutive-reuse counter.
        dl = self.delta[:B, win].reshape(T)
        self.delta[:B, win] = np.where(sel, 0, dl + 1).reshape(B, S_act)

        self.has_prev = True
        self.last_scores = scores
        self.last_idx = idx.astype(np.int32)
        self.last_batch_off = np.searchsorted(idx, np.arange(B + 1) * S_act).astype(np.int32)
        return y.reshape(B, S_act, d)


def scores_only(layer: OracleLayer, x, pos_begin=0):
    """Drift scores that `layer.step(x, ...)` would compute, without touching the state.

    Lines 1-3 of Alg. 1 only; used to check score margins and index sets cheaply.
    """
    x = np.asarray(x, _F)
    B, S_act, d = x.shape
    T = B * S_act
    hd = layer.hd
    xn = rmsnorm(x.reshape(T, d), layer.gain, layer.eps)
    sh = layer.score_head
    q0 = linear(xn, layer.w_q[sh * hd:(sh + 1) * hd])
    if not layer.has_prev:
        return np.full(T, np.inf, _F)
    return drift_score(q0, layer.q_prev[:B, pos_begin:pos_begin + S_act].reshape(T, hd))
