"""Config 4 on a scaled-down stack: the whole decoding trajectory on the GPU against the stack oracle, step by step,
teacher-forced (the oracle adopts the GPU's token choice, and the GPU's refresh decision for the few tokens whose
score lies within the margin of tau, so that both walk the same trajectory and every step is a fresh comparison)."""
import numpy as np
import pytest

from oracle import dare_stack_oracle as sto
from paper_2605_08134_b200 import workloads as wl
from tests import parity

pytestmark = pytest.mark.gpu

# Teacher forcing: a token whose oracle score lies within the margin of tau takes the GPU's refresh decision, so that
# both sides keep walking the same trajectory.  That cannot hide a score error: the tests below check, for every token
# and before anything is adopted, that the GPU's decision is Eq. 2 applied to the GPU's own score, and that this score
# is within the score gate of the oracle's, inside the margin as well as outside.  The margin equals the gate: a score
# closer to tau than the gate may fall on either side by the bf16 rounding of x_norm alone (tests/test_rounding_pins.py).
# Single layer steps from the GPU's own state (full-size test) use the plain bf16 score gate.  Over whole trajectories
# (small stack) the oracle's hidden states are fp64 through all layers while the GPU's pass through bf16 after every
# projection, so the inputs of the deeper layers already differ, and the scores with them: gate and margin are twice
# the single-layer ones there, and the test asserts that the margin decides for fewer than 1 % of the tokens.
SCORE_GATE_LAYER = parity.SCORE_ATOL[wl.DTYPE_BF16]
MARGIN_LAYER = SCORE_GATE_LAYER
SCORE_GATE_STACK = 2 * SCORE_GATE_LAYER
MARGIN_STACK = SCORE_GATE_STACK


def check_gpu_decisions(sel, n_tokens, tau, first, mode):
    """The GPU's refresh list is Eq. 2's complement applied to the GPU's own scores (every token); returns the mask."""
    m = np.zeros(n_tokens, bool)
    m[sel["idx"]] = True
    assert sel["count"] == len(sel["idx"]) and (np.diff(sel["idx"]) > 0).all()
    if first or mode == 0:
        assert m.all()
    else:
        np.testing.assert_array_equal(m, ~(sel["scores"] <= np.float32(tau)))
    return m


@pytest.fixture(scope="module")
def dare():
    from paper_2605_08134_b200 import build
    build.build()
    from paper_2605_08134_b200 import dare as d
    return d


def small_stack(L=4, d=256, H=2, d_ff=768, vocab=1024, prompt=64, gen=64, batch=2):
    lay = wl.scaled(wl.LLADA_LAYER, name="small_stack_layer", d_model=d, n_heads=H, seq=prompt + gen, prompt=prompt,
                    batch=batch, seed=3)
    return wl.StackShape("small_stack", L, lay, d_ff, vocab, gen, seed=3)


def oracle_stack(shape, w, batch):
    lay = shape.layer
    return sto.OracleStack(shape.n_layers, lay.d_model, lay.n_heads, lay.head_dim, shape.d_ff, shape.vocab, batch,
                           lay.seq, lay.rope_theta, lay.rms_eps, w)


@pytest.mark.parametrize("mode,policy", [(3, "fixed"), (1, "fixed"), (3, "first-layers-dense-refresh-every-2nd-step")])
def test_small_stack_decoding_trajectory(dare, mode, policy):
    """policy "fixed": one threshold for every layer and step.  The other one is the schedule of the paper's Fast-dLLM-v2
    experiment (Sec. 5) scaled to four layers: the first layers never reuse, and every second step refreshes
    everything (refresh interval 2); both are per-layer thresholds below zero handed to the step by the caller."""
    import torch
    shape = small_stack()
    lay = shape.layer
    B, P, S = 2, lay.prompt, lay.seq
    w = wl.make_stack_weights(shape)
    base_taus = [0.1] * shape.n_layers
    n_dense_layers = 2
    g = dare.Stack(shape, w, B)
    o = oracle_stack(shape, w, B)
    prompt = wl.random_prompt(shape, B)
    toks_np = np.concatenate([prompt, np.full((B, shape.gen_len), shape.mask_id, np.int32)], axis=1)
    toks = torch.from_numpy(toks_np.copy()).cuda()
    agree = 0
    steps = 0
    near = seen = 0
    reused_rows = 0
    for blk in range(shape.gen_len // lay.block):
        lo, hi = P + blk * lay.block, P + (blk + 1) * lay.block
        for _ in range(lay.block):
            first = steps == 0
            if policy == "fixed":
                taus = base_taus
            elif steps % 2 == 0:
                taus = [-1.0] * shape.n_layers                                   # refresh step: nothing is reused
            else:
                taus = [-1.0] * n_dense_layers + base_taus[n_dense_layers:]      # the first layers never reuse
            pos_begin = 0 if first else P
            S_act = S - pos_begin
            before = toks_np.copy()
            gpos, gtok, gprob = g.decode_step(toks, P, blk, first, mode, taus)
            # the GPU's refresh decisions, per layer, as masks for the oracle to adopt inside the margin
            adopt = []
            gsel = []
            for l in range(shape.n_layers):
                sel = g.layer(l).last_selection(B, S_act)
                m = check_gpu_decisions(sel, B * S_act, taus[l], first, mode)
                adopt.append((m, MARGIN_STACK)); gsel.append(sel)
            hid = o.forward(before[:, pos_begin:], pos_begin, mode, taus, adopt=adopt)
            # (1) refresh sets: identical wherever the oracle's score is clear of tau
            for l in range(shape.n_layers):
                ol = o.layers[l]
                np.testing.assert_array_equal(gsel[l]["idx"], ol.last_idx, err_msg=f"step {steps} layer {l}")
                if taus[l] < 0:
                    assert gsel[l]["count"] == B * S_act                          # a layer told not to reuse refreshes all
                else:
                    reused_rows += B * S_act - gsel[l]["count"]
                if not first:
                    np.testing.assert_allclose(gsel[l]["scores"], ol.last_scores, rtol=0, atol=SCORE_GATE_STACK)
                    near += int((np.abs(ol.last_scores - taus[l]) < MARGIN_STACK).sum())
                    seen += ol.last_scores.size
            # (2) final hidden states of the active rows
            # The states have passed through L layers (each with the bf16 cache roundings that tests/parity.py
            # describes) and a final normalisation to RMS 1: the max-abs gate is the caches' (2 x) times sqrt(L); the
            # RMS gate stays at the plain 2e-2.
            parity.assert_close(f"hidden step {steps}", g.last_hidden(B, S_act), hid, parity.TOL_BF16,
                                max_factor=2.0 * np.sqrt(shape.n_layers))
            # (3) the choice: the GPU's (position, token) must be (near-)optimal under the oracle's probabilities
            for b in range(B):
                cand = np.nonzero(before[b, lo:hi] == shape.mask_id)[0] + lo
                lg = o.logits(hid[b, cand - pos_begin])
                lg[:, shape.mask_id] = -np.inf
                t, p = sto.top1_prob(lg)
                assert gpos[b] in cand and gtok[b] != shape.mask_id
                j = int(np.nonzero(cand == gpos[b])[0][0])
                mx = lg[j].max()
                p_gpu_tok = np.exp(lg[j, gtok[b]] - mx) * p[j]               # oracle probability of the GPU's token
                assert p_gpu_tok >= p.max() * (1 - 5e-2), (steps, b, p_gpu_tok, p.max())
                assert abs(gprob[b] - p_gpu_tok) <= 5e-2 * p_gpu_tok, (steps, b, gprob[b], p_gpu_tok)
                agree += int(cand[int(np.argmax(p))] == gpos[b] and t[j] == gtok[b])
                toks_np[b, gpos[b]] = gtok[b]                                  # teacher forcing: follow the GPU
            np.testing.assert_array_equal(toks.cpu().numpy(), toks_np)
            steps += 1
    assert steps == shape.gen_len and not (toks_np == shape.mask_id).any()
    # With random N(0, 0.02^2) weights the token distribution is nearly flat (top-1 probability ~ 2.4 / vocab), so many
    # candidates tie within bf16 resolution; exact agreement of the arg-max is reported, not required.
    print(f"mode {mode}: {agree} of {steps * B} choices are the oracle's own arg-max")
    assert agree > 0
    assert near < 0.01 * seen, (near, seen)           # the margin decides for a small minority of the tokens only
    assert reused_rows > 0                            # ... and the layers allowed to reuse did
    for l in range(shape.n_layers):
        assert g.layer(l).status() == 0
    g.close()


def test_stack_argument_checks(dare):
    import ctypes as C
    shape = small_stack(L=2)
    cfg_ok = dare.StackConfig(C.sizeof(dare.StackConfig), 2, 768, 1024, 1023, 32,
                              dare.make_config(256, 2, 128, 2, 128, 5e5, 1e-5, dare.BF16))
    assert dare.dare_stack_workspace_bytes(cfg_ok) > 0
    for field, val in (("d_ff", 100), ("vocab", 1000), ("block", 64), ("mask_id", 5000)):
        cfg = dare.StackConfig.from_buffer_copy(cfg_ok)
        setattr(cfg, field, val)
        assert dare.dare_stack_workspace_bytes(cfg) == 0, field
    f32 = dare.StackConfig.from_buffer_copy(cfg_ok)
    f32.layer.dtype = dare.F32
    assert dare.dare_stack_workspace_bytes(f32) == 0
    assert dare.dare_stack_reset(None) == dare.ERR_INVALID_ARG
    assert dare.dare_stack_layer(None, 0) is None


def _torch_stack_weights(shape, torch, seed=3):
    """Full-size weights drawn on the GPU: N(0, 0.02^2) in bf16, gains 1."""
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    d, f, V = shape.layer.d_model, shape.d_ff, shape.vocab
    draw = lambda *dims: (torch.randn(dims, generator=gen, device="cuda") * 0.02).to(torch.bfloat16)
    ones = torch.ones(d, device="cuda")
    w = {"emb": draw(V, d), "head": draw(V, d), "final_gain": ones, "layers": []}
    for _ in range(shape.n_layers):
        w["layers"].append({"w_q": draw(d, d), "w_k": draw(d, d), "w_v": draw(d, d), "w_o": draw(d, d), "rms_gain": ones,
                            "gain2": ones, "w_gate": draw(f, d), "w_up": draw(f, d), "w_down": draw(d, f)})
    return w


def test_full_size_stack_teacher_forced_layer_checks(dare):
    """Config 4 at full size: 32 layers, d 4096, SwiGLU 12288, vocab 126464, 256 prompt + 256 generation positions,
    batch 1, both reuse rules.  The oracle cannot run the whole model, so it checks single layer steps: the state of a
    layer (caches, stored query) and its input are taken from the GPU, one oracle layer step is run from that state,
    and refresh set, caches and the layer's output are compared (tokens whose oracle score lies within the margin of
    tau take the GPU's decision).  The step's token choice is checked against fp64 logits of the GPU's final states."""
    import torch
    from oracle import dare_oracle as orc
    shape = wl.LLADA_STACK
    lay = shape.layer
    P, S, d, B = lay.prompt, lay.seq, lay.d_model, 1
    w = _torch_stack_weights(shape, torch)
    taus = [0.1] * shape.n_layers
    g = dare.Stack(shape, w, B)
    prompt = wl.random_prompt(shape, B)
    toks = torch.from_numpy(np.concatenate([prompt, np.full((B, shape.gen_len), shape.mask_id, np.int32)], axis=1)).cuda()
    checks = {1: (0,), 2: (13,), 5: (31,), 33: (7,)}   # step -> layer checked at that step (33: second block)
    xbuf = torch.empty((B, S - P, d), dtype=torch.bfloat16, device="cuda")
    hbuf = torch.empty_like(xbuf)
    head64 = None
    for step in range(34):
        first = step == 0
        blk = step // lay.block
        layers_now = checks.get(step, ())
        pre = {}
        for l in layers_now[:1]:                         # one captured layer per step
            lv = g.layer(l)
            pre[l] = lv.read_caches(B, S)
            g.set_capture(l, xbuf, hbuf)
        before = toks.cpu().numpy().copy()
        gpos, gtok, gprob = g.decode_step(toks, P, blk, first, 3, taus)
        for l in layers_now[:1]:
            g.set_capture(-1)
            lv = g.layer(l)
            lw = w["layers"][l]
            o = orc.OracleLayer(d, lay.n_heads, lay.head_dim, B, S, lay.rope_theta, lay.rms_eps,
                                *(lw[k].float().cpu().numpy() for k in ("w_q", "w_k", "w_v", "w_o")), np.ones(d))
            o.has_prev, o.batch, o.kv_len = True, B, S
            o.q_prev[:] = pre[l]["q_prev"]; o.k_cache[:] = pre[l]["k"]; o.v_cache[:] = pre[l]["v"]; o.o_cache[:] = pre[l]["o"]
            sel = lv.last_selection(B, S - P)
            gm = check_gpu_decisions(sel, S - P, taus[l], False, 3)
            x = xbuf.float().cpu().numpy()
            y = o.step(x, 3, taus[l], pos_begin=P, adopt=(gm, MARGIN_LAYER))
            np.testing.assert_array_equal(sel["idx"], o.last_idx, err_msg=f"step {step} layer {l}")
            np.testing.assert_allclose(sel["scores"], o.last_scores, rtol=0, atol=SCORE_GATE_LAYER)
            assert 1 <= sel["count"] <= 8                # one new token per step: a handful of refreshed rows at most
            parity.assert_close(f"h step {step} layer {l}", hbuf.float().cpu().numpy(), x + y, parity.TOL_BF16)
            post = lv.read_caches(B, S)
            parity.assert_close("k_cache", post["k"], o.k_cache, parity.TOL_BF16, max_factor=2.0)
            parity.assert_close("v_cache", post["v"], o.v_cache, parity.TOL_BF16, max_factor=2.0)
            parity.assert_close("o_cache", post["o"], o.o_cache, parity.TOL_BF16, max_factor=2.0)
            # rows outside the refresh set: untouched, bit for bit (Eq. 3, Eq. 4)
            keep = np.ones(S, bool); keep[P + sel["idx"]] = False
            assert np.array_equal(post["k"][0, keep], pre[l]["k"][0, keep])
            assert np.array_equal(post["o"][0, keep], pre[l]["o"][0, keep])
        if step in (0, 2, 33):
            # the choice under fp64 logits of the GPU's own final states
            if head64 is None:
                head64 = w["head"].float().cpu().numpy().astype(np.float64)
            pos_begin = 0 if first else P
            hid = g.last_hidden(B, S - pos_begin)
            lo = P + blk * lay.block
            cand = np.nonzero(before[0, lo:lo + lay.block] == shape.mask_id)[0] + lo
            lg = hid[0, cand - pos_begin].astype(np.float64) @ head64.T
            lg[:, shape.mask_id] = -np.inf
            t, p = sto.top1_prob(lg)
            j = int(np.nonzero(cand == gpos[0])[0][0])
            p_tok = np.exp(lg[j, gtok[0]] - lg[j].max()) * p[j]
            assert p_tok >= p.max() * (1 - 2e-2), (step, p_tok, p.max())
            assert abs(gprob[0] - p_tok) <= 2e-2 * p_tok
    assert not (toks[:, P:P + 32] == shape.mask_id).any() and (toks[:, P + 34:] == shape.mask_id).all()
    for l in (0, 13, 31):
        assert g.layer(l).status() == 0
    g.close()


def test_decode_steps_replay_from_cuda_graphs(dare):
    """The decode step takes no decision on the host: one capture per block, replayed for the block's tokens, generates
    the same tokens as the same steps enqueued one by one."""
    import torch
    shape = small_stack()
    lay = shape.layer
    B, P = 2, lay.prompt
    w = wl.make_stack_weights(shape)
    taus = [0.1] * shape.n_layers
    prompt = wl.random_prompt(shape, B)
    start = np.concatenate([prompt, np.full((B, shape.gen_len), shape.mask_id, np.int32)], axis=1)
    n_steps = shape.gen_len // 2                       # per sequence one token per step: half of the generation

    direct = dare.Stack(shape, w, B)
    toks_d = torch.from_numpy(start.copy()).cuda()
    picks_d = []
    for step in range(n_steps):
        picks_d.append(direct.decode_step(toks_d, P, step // lay.block, step == 0, 3, taus))

    graphed = dare.Stack(shape, w, B)
    toks_g = torch.from_numpy(start.copy()).cuda()
    res = tuple(torch.empty(B, dtype=t, device="cuda") for t in (torch.int32, torch.int32, torch.float32))
    graphed.decode_step_enqueue(toks_g, P, 0, True, 3, taus, out=res)
    graphed.decode_step_enqueue(toks_g, P, 0, False, 3, taus, out=res)     # every kernel of a window step has run once
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    step = 2
    while step < n_steps:
        blk = step // lay.block
        n_here = min(n_steps, (blk + 1) * lay.block) - step
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            graphed.decode_step_enqueue(toks_g, P, blk, False, 3, taus, out=res)
        for i in range(n_here):
            graph.replay()
            torch.cuda.synchronize()
            pos, tok, prob = (r.cpu().numpy() for r in res)
            np.testing.assert_array_equal(pos, picks_d[step + i][0])
            np.testing.assert_array_equal(tok, picks_d[step + i][1])
            np.testing.assert_array_equal(prob, picks_d[step + i][2])
        step += n_here
    assert torch.equal(toks_g, toks_d)
    direct.close(); graphed.close()
