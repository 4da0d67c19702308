"""fp64 CPU oracle for a stack of DARE attention layers inside a pre-norm transformer (config 4).

TEST INFRASTRUCTURE ONLY: same rules as dare_oracle.py (never imported by the product).

The paper describes DARE as a plug-in to an existing diffusion-LLM stack and defines only the attention layer
(Alg. 1, Alg. 2); its appendix model is one layer with a generic MLP (Appendix E.1).  For a 32-layer LLaDA-shaped
stack the surrounding block is read as the usual pre-norm residual block:

    h   = x + Attn_DARE(x)                      Attn_DARE = dare_oracle.OracleLayer.step (it normalises x itself)
    out = h + W_D ( silu(W_G n) * (W_U n) )     n = RMSNorm_2(h)       (SwiGLU; MLP dense on every active row,
                                                                        Appendix E.1 applies the MLP to all rows)
then a final RMSNorm and an untied LM head.  Decoding (Appendix A: block size 32, generation length 256) is read as:
step 0 runs the whole sequence (prompt + masked generation positions) and fills every cache; afterwards only the
generation window is active and the prompt's K/V rows stay frozen (prefix cache); every step un-masks, inside the
active 32-token block, the one masked position whose top-1 softmax probability is largest (lowest index on ties),
greedily; blocks go left to right.
"""
from __future__ import annotations

import numpy as np

from . import dare_oracle as orc

_F = np.float64


def silu(x):
    x = np.asarray(x, _F)
    return x / (1.0 + np.exp(-x))


def swiglu_mlp(n, w_gate, w_up, w_down):
    """W_D ( silu(W_G n) * (W_U n) ), weights stored [out, in]."""
    return orc.linear(silu(orc.linear(n, w_gate)) * orc.linear(n, w_up), w_down)


def top1_prob(logits):
    """(argmax, softmax probability of the argmax) per row; lowest index on ties."""
    logits = np.asarray(logits, _F)
    tok = np.argmax(logits, axis=-1)
    mx = np.max(logits, axis=-1, keepdims=True)
    p = 1.0 / np.sum(np.exp(logits - mx), axis=-1)
    return tok, p


class OracleStack:
    def __init__(self, n_layers, d_model, n_heads, head_dim, d_ff, vocab, max_batch, max_seq, rope_theta, rms_eps,
                 weights):
        """weights: dict(emb [V,d], head [V,d], final_gain [d], layers=[dict(w_q,w_k,w_v,w_o,rms_gain, gain2,
        w_gate [d_ff,d], w_up [d_ff,d], w_down [d,d_ff])])"""
        self.L, self.d, self.V, self.eps = n_layers, d_model, vocab, float(rms_eps)
        self.emb = np.asarray(weights["emb"], _F)
        self.head = np.asarray(weights["head"], _F)
        self.final_gain = np.asarray(weights["final_gain"], _F)
        self.lw = weights["layers"]
        self.layers = [orc.OracleLayer(d_model, n_heads, head_dim, max_batch, max_seq, rope_theta, rms_eps,
                                       lw["w_q"], lw["w_k"], lw["w_v"], lw["w_o"], lw["rms_gain"]) for lw in self.lw]
        self.layer_inputs = None

    def reset(self):
        for l in self.layers:
            l.reset()

    def forward(self, tokens, pos_begin, mode, taus, keep_inputs=False, adopt=None):
        """tokens: int [B, S_act] at positions [pos_begin, pos_begin+S_act).  Returns the final-normed hidden states
        [B, S_act, d].  taus: one threshold per layer.  adopt: per layer, the (mask, margin) of OracleLayer.step."""
        tokens = np.asarray(tokens)
        x = self.emb[tokens]
        self.layer_inputs = [] if keep_inputs else None
        for l, (layer, lw) in enumerate(zip(self.layers, self.lw)):
            if keep_inputs:
                self.layer_inputs.append(x.copy())
            a = layer.step(x, mode, taus[l], pos_begin=pos_begin, adopt=None if adopt is None else adopt[l])
            h = x + a
            n = orc.rmsnorm(h, lw["gain2"], self.eps)
            x = h + swiglu_mlp(n, lw["w_gate"], lw["w_up"], lw["w_down"])
        return orc.rmsnorm(x, self.final_gain, self.eps)

    def logits(self, hidden_rows):
        return orc.linear(hidden_rows, self.head)


def generate(stack: OracleStack, prompt_ids, gen_len, block, mask_id, mode, taus, forced=None):
    """Block-wise greedy decoding of one batch of sequences (all share the prompt length).

    prompt_ids: int [B, P].  Returns (tokens [B, P+gen_len], trace) where trace[k] = dict(step, pos [B], tok [B],
    prob [B]) for every un-masking step.  `forced`, if given, is a list of (pos [B], tok [B]) per step that
    overrides the oracle's own choice (teacher forcing when comparing with another implementation).
    """
    prompt_ids = np.asarray(prompt_ids)
    B, P = prompt_ids.shape
    S = P + gen_len
    tokens = np.concatenate([prompt_ids, np.full((B, gen_len), mask_id, prompt_ids.dtype)], axis=1)
    trace = []
    stack.reset()
    step = 0
    for blk in range(gen_len // block):
        lo, hi = P + blk * block, P + (blk + 1) * block
        for _ in range(block):
            if step == 0:
                hidden = stack.forward(tokens, 0, mode, taus)             # whole sequence: fills every cache
                off = 0
            else:
                hidden = stack.forward(tokens[:, P:], P, mode, taus)      # generation window only
                off = P
            pos = np.zeros(B, int); tok = np.zeros(B, int); prob = np.zeros(B)
            for b in range(B):
                cand = np.nonzero(tokens[b, lo:hi] == mask_id)[0] + lo
                lg = stack.logits(hidden[b, cand - off])
                lg[:, mask_id] = -np.inf                                  # the mask token itself is never emitted
                t, p = top1_prob(lg)
                j = int(np.argmax(p))                                     # first maximum: lowest index on ties
                pos[b], tok[b], prob[b] = cand[j], t[j], p[j]
            trace.append({"step": step, "pos": pos.copy(), "tok": tok.copy(), "prob": prob.copy()})
            if forced is not None:
                pos, tok = forced[step]
            for b in range(B):
                tokens[b, pos[b]] = tok[b]
            step += 1
    return tokens, trace
