"""Seeded synthetic inputs for the DARE layer step.

This module only draws numbers and formats them; it holds none of the method's
arithmetic (no norm, projection, score or attention) so that both the CUDA path
and the independent CPU oracle can be fed the very same arrays.

The workloads stand in for the paper's measurements on trained LLaDA/Dream
weights and public benchmark suites (Appendix A), which need data that is not
available offline.  What is kept is their shape and structure: the LLaDA-8B layer
geometry, block size 32 and generation length 256 (Appendix A), a drift-score
distribution with a strong near-zero mode (Sec. 5, per-token drift figure), change
concentrated in the active block, and reuse of up to 87 % (abstract).

All draws are float32 from numpy's default_rng(seed) and are then rounded to the
layer's storage type (round-to-nearest-even for bf16).  Hidden states keep a
float32 master copy across steps: noise and redraws are applied to the master and
a rounded copy is handed out.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

DTYPE_F32 = 0
DTYPE_BF16 = 1


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(a, np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float32 (exact)."""
    return (np.ascontiguousarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32)


def bf16_round(a: np.ndarray) -> np.ndarray:
    """float32 values rounded to the nearest bf16-representable float32."""
    return bf16_bits_to_f32(bf16_bits(a)).reshape(np.shape(a))


def round_to(a: np.ndarray, dtype: int) -> np.ndarray:
    a = np.ascontiguousarray(a, np.float32)
    return bf16_round(a) if dtype == DTYPE_BF16 else a


@dataclass(frozen=True)
class LayerShape:
    name: str
    d_model: int
    n_heads: int
    head_dim: int
    batch: int
    seq: int
    prompt: int              # leading positions that belong to the prompt
    rope_theta: float
    dtype: int
    rms_eps: float = 1e-5
    block: int = 32
    seed: int = 0

    @property
    def tokens(self) -> int:
        return self.batch * self.seq


# The five benchmark configurations (layer geometry only).
TINY_F32 = LayerShape("tiny_f32", 256, 4, 64, 1, 128, 64, 1e4, DTYPE_F32, seed=0)
LLADA_LAYER = LayerShape("llada8b_layer_b1_s512", 4096, 32, 128, 1, 512, 256, 5e5, DTYPE_BF16, seed=1)
LLADA_DARE_O = LayerShape("llada8b_layer_b8_s1024", 4096, 32, 128, 8, 1024, 512, 5e5, DTYPE_BF16, seed=2)
LLADA_LONG = LayerShape("llada8b_layer_b4_s4096", 4096, 32, 128, 4, 4096, 2048, 5e5, DTYPE_BF16, seed=4)


def scaled(shape: LayerShape, **kw) -> LayerShape:
    """A copy of `shape` with some fields replaced (reduced cases for CPU-checkable parity)."""
    d = dict(shape.__dict__)
    d.update(kw)
    return LayerShape(**d)


def make_weights(shape: LayerShape, seed: int | None = None, std: float = 0.02) -> dict:
    """W_Q, W_K, W_V, W_O ~ N(0, std^2), stored [out, in]; unit RMSNorm gain."""
    rng = np.random.default_rng((shape.seed if seed is None else seed) + 7919)
    d = shape.d_model
    w = {}
    for name in ("w_q", "w_k", "w_v", "w_o"):
        w[name] = round_to(rng.standard_normal((d, d), dtype=np.float32) * np.float32(std), shape.dtype)
    w["rms_gain"] = np.ones(d, np.float32)
    return w


def uniform_positions(rng, shape: LayerShape, count_per_seq: int) -> np.ndarray:
    """`count_per_seq` distinct positions per sequence, uniform over the sequence. -> bool [B, S]."""
    m = np.zeros((shape.batch, shape.seq), bool)
    for b in range(shape.batch):
        m[b, rng.choice(shape.seq, size=count_per_seq, replace=False)] = True
    return m


def clustered_positions(rng, shape: LayerShape, step: int, clustered_per_seq: int,
                        scattered_per_seq: int, steps_per_block: int = 4) -> np.ndarray:
    """Changed positions concentrated at the active generation block.

    A contiguous run of `clustered_per_seq` positions starts at the first position of the active
    block (block index = step // steps_per_block, wrapping inside the generation region; a run
    that would pass the end of the sequence wraps to the start of the generation region, and one
    longer than the generation region wraps over the whole sequence) plus
    `scattered_per_seq` positions uniform over the remaining ones.  -> bool [B, S].
    """
    gen = shape.seq - shape.prompt
    n_blocks = max(1, gen // shape.block)
    start = ((step // steps_per_block) % n_blocks) * shape.block
    m = np.zeros((shape.batch, shape.seq), bool)
    if clustered_per_seq <= gen:
        run = shape.prompt + (start + np.arange(clustered_per_seq)) % gen
    else:       # a run longer than the generation region goes on through the whole sequence
        run = (shape.prompt + start + np.arange(clustered_per_seq)) % shape.seq
    for b in range(shape.batch):
        m[b, run] = True
        rest = np.nonzero(~m[b])[0]
        if scattered_per_seq:
            m[b, rng.choice(rest, size=scattered_per_seq, replace=False)] = True
    return m


@dataclass
class HiddenStream:
    """Hidden states of consecutive denoising steps for one layer.

    `first()` draws x ~ N(0,1).  `advance(changed)` redraws the rows flagged in `changed`
    from N(0,1) and adds N(0, noise_std^2) to all other rows (std, not variance).
    """
    shape: LayerShape
    seed: int | None = None
    noise_std: float = 1e-3
    master: np.ndarray = field(init=False, default=None)

    def __post_init__(self):
        s = self.shape.seed if self.seed is None else self.seed
        self.rng = np.random.default_rng(s)

    def first(self) -> np.ndarray:
        sh = self.shape
        self.master = self.rng.standard_normal((sh.batch, sh.seq, sh.d_model), dtype=np.float32)
        return round_to(self.master, sh.dtype)

    def advance(self, changed: np.ndarray) -> np.ndarray:
        sh = self.shape
        changed = np.asarray(changed, bool).reshape(sh.batch, sh.seq)
        noise = self.rng.standard_normal(self.master.shape, dtype=np.float32) * np.float32(self.noise_std)
        fresh = self.rng.standard_normal(self.master.shape, dtype=np.float32)
        self.master = np.where(changed[:, :, None], fresh, self.master + noise)
        return round_to(self.master, sh.dtype)

    def advance_graded(self, lo: float = 1e-3, hi: float = 1.0) -> np.ndarray:
        """Every row gets noise whose std is log-uniform in [lo, hi]: scores spread over decades."""
        sh = self.shape
        std = np.exp(self.rng.uniform(np.log(lo), np.log(hi), size=(sh.batch, sh.seq, 1))).astype(np.float32)
        noise = self.rng.standard_normal(self.master.shape, dtype=np.float32) * std
        self.master = self.master + noise
        return round_to(self.master, sh.dtype)


def two_step_case(shape: LayerShape, changed_per_seq: int, seed: int | None = None):
    """(weights, x0, x1, changed mask) for the basic two-step test: uniform changed positions."""
    w = make_weights(shape, seed)
    hs = HiddenStream(shape, seed)
    x0 = hs.first()
    changed = uniform_positions(hs.rng, shape, changed_per_seq)
    x1 = hs.advance(changed)
    return w, x0, x1, changed


@dataclass(frozen=True)
class StackShape:
    """A stack of DARE attention layers inside pre-norm SwiGLU blocks (config 4 geometry or a reduced copy)."""
    name: str
    n_layers: int
    layer: LayerShape          # attention geometry; layer.seq = prompt + generation length, layer.prompt = prompt
    d_ff: int
    vocab: int
    gen_len: int
    seed: int = 3

    @property
    def mask_id(self) -> int:
        return self.vocab - 1


LLADA_STACK = StackShape("llada8b_stack_32l", 32, scaled(LLADA_LAYER, name="llada8b_stack_layer", seed=3),
                         12288, 126464, 256)


def make_stack_weights(shape: StackShape, seed: int | None = None, std: float = 0.02) -> dict:
    """All matrices ~ N(0, std^2) rounded to the storage type, gains 1: embedding [V, d], untied head [V, d], and per
    layer W_Q, W_K, W_V, W_O [d, d], W_gate, W_up [d_ff, d], W_down [d, d_ff]."""
    s = shape.seed if seed is None else seed
    rng = np.random.default_rng(s + 104729)
    lay, d, f = shape.layer, shape.layer.d_model, shape.d_ff
    draw = lambda *dims: round_to(rng.standard_normal(dims, dtype=np.float32) * np.float32(std), lay.dtype)
    w = {"emb": draw(shape.vocab, d), "head": draw(shape.vocab, d), "final_gain": np.ones(d, np.float32), "layers": []}
    for _ in range(shape.n_layers):
        w["layers"].append({"w_q": draw(d, d), "w_k": draw(d, d), "w_v": draw(d, d), "w_o": draw(d, d),
                            "rms_gain": np.ones(d, np.float32), "gain2": np.ones(d, np.float32),
                            "w_gate": draw(f, d), "w_up": draw(f, d), "w_down": draw(d, f)})
    return w


def random_prompt(shape: StackShape, batch: int, seed: int | None = None) -> np.ndarray:
    """`prompt` random token ids per sequence, never the mask id."""
    rng = np.random.default_rng((shape.seed if seed is None else seed) + 31)
    return rng.integers(0, shape.vocab - 1, size=(batch, shape.layer.prompt), dtype=np.int32)
