#!/usr/bin/env python
"""Benchmark of the DARE layer step (per-layer latency and token-positions per second).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--mode both|kv|o|dense]
                    [--changed 0.13] [--layers 8]

One "step" = one `dare_layer_step` = the whole hot path (norm, Q projection + drift score, threshold +
compaction, gathered K/V projection + cache scatter, row-sparse attention, output projection) over one batch.
Workload at N = 1: the LLaDA-8B-shaped attention layer, batch 1, seq 512, bf16, 13 % of the tokens changed per
step (87 % reuse), mode "both".  Steps rotate over `--layers` layer instances (8 x 134 MB of weights, far more than
the 126 MB L2) and alternate between two hidden-state buffers so that every timed step refreshes the same
planned token set.

Timing: after W warm-up steps the region of exactly K steps (barrier + synchronise on both sides, CUDA events, max over
ranks) is repeated until at least a second of it has been timed; `ms_per_step` is the median over the repeats, p10 / p90
and the number of repeats go with it.  The dense path and the end-to-end figure follow the same protocol.

Prints ONE JSON line.  `--impl reference` times the fp64 CPU oracle on the same workload instead.  `--gpus N` with
N > 1 and no torchrun environment starts N ranks itself (one replica per GPU).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

MODES = {"dense": 0, "kv": 1, "o": 2, "both": 3}
TAU = 0.1


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            try:
                pw.append(float(r[2]))
            except ValueError:
                pass
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "power_w_max": max(pw) if pw else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def workload_config(shape, args, n_refreshed, world):
    """The `config` object of the JSON line: the workload and how the timed steps see HBM; both arms print the same."""
    d = shape.d_model
    return {"workload": shape.name, "d_model": d, "n_heads": shape.n_heads, "head_dim": shape.head_dim,
            "batch": shape.batch, "seq_len": shape.seq, "mode": args.mode, "changed_fraction": args.changed,
            "refreshed_tokens": int(n_refreshed), "threshold": TAU, "layers_rotated": args.layers,
            "l2": "inputs larger than L2: weights of %d layer instances (%.0f MB) rotate"
                  % (args.layers, args.layers * 4 * d * d * 2 / 1e6),
            "parallelism": "replicas" if world > 1 else "single"}


def percentiles(values):
    """(median, p10, p90) of a list of per-step times."""
    v = sorted(values)
    pick = lambda q: v[min(len(v) - 1, max(0, int(round(q * (len(v) - 1)))))]
    return statistics.median(v), pick(0.10), pick(0.90)


def load_traffic(workload):
    """DRAM bytes per launch and kernel from the ncu capture summarised under profiles/ (None when there is none)."""
    path = os.path.join(ROOT, "profiles", f"dram_traffic_{workload}_both13.json")
    try:
        with open(path) as f:
            return json.load(f)
    except OSError:
        return None


def make_inputs_np(shape, changed_frac, seed):
    """Two hidden-state buffers A, B: B redraws `changed_frac` of the rows of A (uniform positions) and perturbs the
    rest by N(0, (1e-3)^2) before bf16 rounding; stepping A -> B -> A ... refreshes the same set every time."""
    from paper_2605_08134_b200 import workloads as wl
    hs = wl.HiddenStream(shape, seed)
    xa = hs.first()
    n = int(round(changed_frac * shape.seq))
    changed = wl.uniform_positions(hs.rng, shape, n)      # n positions in every sequence
    xb = hs.advance(changed)
    return xa, xb, changed


def make_inputs(shape, changed_frac, seed, torch, device):
    import numpy as np
    xa, xb, changed = make_inputs_np(shape, changed_frac, seed)
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device).to(torch.bfloat16)
    return xa, xb, changed, to(xa), to(xb)


def make_layers(shape, n_layers, seed, torch, device, dare):
    layers = []
    gen = torch.Generator(device=device)
    for l in range(n_layers):
        gen.manual_seed(seed * 1000 + l)
        w = {k: (torch.randn((shape.d_model, shape.d_model), generator=gen, device=device, dtype=torch.float32) * 0.02)
             .to(torch.bfloat16) for k in ("w_q", "w_k", "w_v", "w_o")}
        w["rms_gain"] = torch.ones(shape.d_model, device=device, dtype=torch.float32)
        layers.append(dare.Layer(shape, w, device=device))
    return layers


def run_ours(args):
    import numpy as np
    import torch
    from paper_2605_08134_b200 import build
    build.build()
    from paper_2605_08134_b200 import dare, distrib, workloads as wl

    rank, local_rank, world = distrib.rank_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    shape = wl.LLADA_LAYER
    if args.d_model or args.seq or args.batch:      # exploration only: the reported workload is the default one
        dm = args.d_model or shape.d_model
        sq = args.seq or shape.seq
        shape = wl.scaled(shape, name=f"custom_d{dm}_b{args.batch or shape.batch}_s{sq}", d_model=dm,
                          n_heads=dm // shape.head_dim, seq=sq, prompt=sq // 2, batch=args.batch or shape.batch)
    mode = MODES[args.mode]
    peaks = load_peaks()
    # every rank runs its own replica (sequences are independent: batch sharding, no data-path collective)
    xa_np, xb_np, changed, xa, xb = make_inputs(shape, args.changed, distrib.rank_seed(shape.seed, rank), torch, device)
    n_planned = int(changed.sum())
    layers = make_layers(shape, args.layers, shape.seed + 17 * rank, torch, device, dare)
    y = torch.empty_like(xa)
    stream = torch.cuda.current_stream(device)
    T = shape.tokens

    def one_pass(steps, m, start_parity=0, host=None, pipelined=False):
        launches = 0
        for i in range(steps):
            lay = layers[i % len(layers)]
            # the parity of a layer's own step count decides which buffer it sees next
            k = lay._bench_steps
            src = (xa, xb)[k & 1] if host is None else host[k & 1]
            if host is None:
                lay.step(src, m, TAU, y)
            elif pipelined:
                lay.step_host_async(src, m, TAU, host[2][i % len(layers)])
            else:
                lay.step_host(src, m, TAU, host[2][0])
            lay._bench_steps = k + 1
            launches += lay.launch_count()
        if pipelined:
            for lay in layers:
                lay.wait_host()
        return launches

    def prime(m):
        for lay in layers:
            lay.reset()
            lay._bench_steps = 0
        one_pass(len(layers), m)          # first step of every layer is dense and fills its caches
        torch.cuda.synchronize()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def timed_once(steps, m, host=None, pipelined=False):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0 = time.perf_counter()
        ev0.record(stream)
        launches = one_pass(steps, m, host=host, pipelined=pipelined)
        ev1.record(stream)
        torch.cuda.synchronize()
        wall = time.perf_counter() - t0
        dev_ms = ev0.elapsed_time(ev1)
        ms = wall * 1e3 if host is not None else dev_ms
        ms = distrib.max_over_ranks(ms, dist, device)
        barrier()
        return ms, launches

    def timed(steps, m, host=None, pipelined=False, min_total_ms=1000.0, max_repeats=4000):
        """The K-step region repeated until `min_total_ms` of it have been timed (every rank sees the same max-over-ranks
        times, so all stop together).  -> per-step times of the repeats (ms), launches of one region."""
        per_step, total, launches = [], 0.0, 0
        while True:
            ms, launches = timed_once(steps, m, host=host, pipelined=pipelined)
            per_step.append(ms / steps)
            total += ms
            if total >= min_total_ms or len(per_step) >= max_repeats:
                return per_step, launches

    # ---- reuse path: warm-up, then regions of exactly K timed steps with the clocks sampled
    prime(mode)
    one_pass(max(args.warmup, 3), mode)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    reuse_times, launches = timed(args.steps, mode, min_total_ms=args.min_ms)
    clocks = sampler.stop() if rank == 0 else None
    ms_per_step, ms_p10, ms_p90 = percentiles(reuse_times)
    # selection really is the planned one
    sel = layers[0].last_selection(shape.batch, shape.seq)
    expect = T if mode == 0 else n_planned
    assert sel["count"] == expect, (sel["count"], expect)
    if mode != 0:
        assert np.array_equal(sel["idx"], np.nonzero(changed.reshape(-1))[0])
    assert all(l.status() == 0 for l in layers)

    # ---- dense path of the same library, same protocol
    prime(0)
    one_pass(max(args.warmup, 3), 0)
    dense_sampler = ClockSampler(local_rank)
    if rank == 0:
        dense_sampler.start()
        time.sleep(0.15)
    dense_times, _ = timed(args.steps, 0, min_total_ms=args.min_ms)
    dense_clocks = dense_sampler.stop() if rank == 0 else None
    dense_ms_per_step, dense_p10, dense_p90 = percentiles(dense_times)

    # ---- per-kernel times: a second pass of K steps with an event before every kernel
    prime(mode)
    one_pass(max(args.warmup, 3), mode)
    for lay in layers:
        lay.set_profiling(True)
    acc = {}
    barrier()
    for i in range(args.steps):
        lay = layers[i % len(layers)]
        k = lay._bench_steps
        lay.step((xa, xb)[k & 1], mode, TAU, y)
        lay._bench_steps = k + 1
        for name, ms in lay.kernel_times():
            acc.setdefault(name, []).append(ms)
    for lay in layers:
        lay.set_profiling(False)
    kernels = {k: 1e3 * sum(v) / len(v) for k, v in acc.items()}          # microseconds per launch

    # ---- the same kernels inside the undisturbed chain: device timestamps (%globaltimer) written by the kernels
    # themselves, from the return of a kernel's wait on its predecessor to the exit of its last CTA.  The events of
    # the pass above break the programmatic launch overlap and add a few microseconds to every kernel; these do not.
    in_chain = {}
    if not args.no_in_chain:
        try:
            one_pass(2 * len(layers), mode)
            for lay in layers:
                lay.debug_timestamps(True)
            one_pass(4 * len(layers), mode)
            torch.cuda.synchronize()
            acc2 = {}
            for lay in layers:
                ts = lay.debug_timestamps(False).astype(np.int64)
                q, kv, at, out = ts[0], ts[1], ts[2], ts[3]
                if min(q[1], kv[1], out[1], at[0]) <= 0:
                    continue
                for name, us in (("q_gemm", (q[6] - q[1]) / 1e3), ("kv_gemm", (kv[6] - kv[1]) / 1e3),
                                 ("attention", (at[6] - max(at[0], kv[6])) / 1e3), ("out_gemm", (out[6] - out[1]) / 1e3)):
                    if 0 < us < 1e6:
                        acc2.setdefault(name, []).append(us)
            in_chain = {k: sum(v) / len(v) for k, v in acc2.items()}
        except Exception:                 # diagnostics only: the bench line stands without them
            in_chain = {}
        barrier()

    # ---- the same steps replayed from a CUDA graph (two steps of every layer instance captured once): what a caller
    # gains by taking the launches off the host.  Diagnostics only; `value` stays the stream-launched number.
    # (no collective inside the try: a rank whose capture failed must still meet the others at the same barriers)
    graph_local = -1.0
    try:
        prime(mode)
        one_pass(max(args.warmup, 3), mode)
        torch.cuda.synchronize()
        n_cap = 2 * len(layers)
        graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream(device)
        with torch.cuda.graph(graph, stream=side):
            one_pass(n_cap, mode)
        reps = max(1, args.steps // n_cap)
        for _ in range(3):
            graph.replay()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ev0.record(stream)
        for _ in range(reps):
            graph.replay()
        ev1.record(stream)
        torch.cuda.synchronize()
        sel = layers[0].last_selection(shape.batch, shape.seq)
        assert sel["count"] == expect and all(l.status() == 0 for l in layers)
        graph_local = ev0.elapsed_time(ev1) / (reps * n_cap)
        del graph
    except Exception as e:                # diagnostics only
        print(f"graph replay not measured: {e!r}", file=sys.stderr)
        graph_local = -1.0
    barrier()
    # slowest rank's figure; dropped if any rank has none
    graph_failed = distrib.max_over_ranks(1.0 if graph_local < 0 else 0.0, dist, device) > 0
    graph_ms_per_step = distrib.max_over_ranks(graph_local, dist, device)
    if graph_failed:
        graph_ms_per_step = None

    # ---- end to end through the host-buffer entry point (pinned host x and y, copies inside the timed region)
    prime(mode)
    xh = [torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).pin_memory() for a in (xa_np, xb_np)]
    yh = [torch.empty_like(xh[0]).pin_memory() for _ in layers]          # one result buffer per layer instance
    one_pass(max(args.warmup, 3), mode, host=(xh[0], xh[1], yh))
    sync_times, _ = timed(args.steps, mode, host=(xh[0], xh[1], yh), min_total_ms=args.min_ms / 4)
    e2e_sync_ms_per_step = percentiles(sync_times)[0]
    # ... and through the enqueue-only entry point: a layer's copy in, step and copy out run on three streams, so the
    # copies of one layer instance overlap the kernels of another (every step still copies its 4 MB in and out).
    # A region of K steps that starts and ends drained does not fill that pipeline when K is small, so two figures are
    # taken: the K-step region as it is (median over the repeats), and regions long enough to run full (a tenth of the
    # time budget each, ten of them): the second is what a caller who keeps stepping sees and is the one reported as
    # `e2e.value`.
    prime(mode)
    one_pass(max(args.warmup, 3), mode, host=(xh[0], xh[1], yh), pipelined=True)
    drained_times, _ = timed(args.steps, mode, host=(xh[0], xh[1], yh), pipelined=True, min_total_ms=args.min_ms / 4)
    e2e_drained_ms = percentiles(drained_times)[0]
    long_steps = max(args.steps, int(math.ceil(args.min_ms / 10.0 / e2e_drained_ms / len(layers))) * len(layers))
    long_times = [timed_once(long_steps, mode, host=(xh[0], xh[1], yh), pipelined=True)[0] / long_steps for _ in range(10)]
    e2e_ms_per_step, e2e_p10, e2e_p90 = percentiles(long_times)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (algorithmic work of the DARE step itself, never the dense work avoided)
    d, n = shape.d_model, (n_planned if mode != 0 else T)
    n_kv = n if (mode & 1) else T
    n_o = n if (mode & 2) else T
    # algorithmic work per launch (what the DARE step itself must move or compute, never the dense work avoided):
    #   projections: 2*M*d*d flop each; the K/V projection of a small refresh set is a stream of both weight
    #   matrices (2*d*d*2 bytes) plus the gathered rows in and the K, V rows out (3*n*d*2 bytes); with many tokens
    #   (more than eight 128-row tiles) a step that reuses attention outputs projects only the refresh set's rows
    #   through W_O (its slot then also holds the copy of the reused rows);
    #   attention: 4*rows*S*d flop; RMSNorm: read + write of [T, d] bf16; selection: scores in, staleness counters
    #   in and out, index list out.
    many = shape.batch * ((shape.seq + 127) // 128) > 8
    n_out = n if ((mode & 2) and many) else T
    work = {
        "q_gemm": ("tensor", 2.0 * T * d * d),
        "out_gemm": ("tensor", 2.0 * n_out * d * d),
        "kv_gemm": ("hbm", 2.0 * d * d * 2 + 3.0 * n_kv * d * 2) if n_kv <= 215 else ("tensor", 4.0 * n_kv * d * d),
        "attention": ("tensor", 4.0 * n_o * shape.seq * d),   # n_o counts rows of all sequences
        "rmsnorm": ("hbm", 2.0 * T * d * 2),
        "select_compact": ("hbm", 12.0 * T + 4.0 * n),
    }
    rows = []
    for name, us in kernels.items():
        if name in work and us > 0:
            bound, amount = work[name]
            if bound == "hbm":
                ach, peak, unit = amount / (us * 1e-6) / 1e9, peaks["hbm_gbs"], "GB/s"
            else:
                ach, peak, unit = amount / (us * 1e-6) / 1e12, peaks["bf16_tflops_sustained"], "TFLOP/s"
            rows.append({"kernel": name, "us": round(us, 2), "bound": bound, "achieved": round(ach, 1), "peak": peak,
                         "unit": unit, "frac": round(ach / peak, 4)})
            if name in in_chain:
                scale = 1e9 if bound == "hbm" else 1e12
                rows[-1]["in_chain"] = {"us": round(in_chain[name], 2),
                                        "achieved": round(amount / (in_chain[name] * 1e-6) / scale, 1),
                                        "frac": round(amount / (in_chain[name] * 1e-6) / scale / peak, 4)}
        else:
            rows.append({"kernel": name, "us": round(us, 2)})
    dom = max((r for r in rows if "bound" in r), key=lambda r: r["us"])
    # DRAM bytes per launch of every kernel from the ncu capture of this workload summarised under profiles/
    traffic = (load_traffic(shape.name) or {}) if (mode == 3 and abs(args.changed - 0.13) < 1e-9) else {}
    for r in rows:
        t = traffic.get("dram_bytes_per_launch", {}).get(r["kernel"])
        if t is not None:
            r["traffic"] = t
    roofline = {"kernel": dom["kernel"], "bound": dom["bound"], "achieved": dom["achieved"], "peak": dom["peak"],
                "unit": dom["unit"], "frac": dom["frac"],
                "traffic": traffic.get("dram_bytes_per_launch", {}).get(dom["kernel"]),
                "traffic_source": traffic.get("source"),
                "peak_source": f"of {peaks['source']} (sustained figure: the kernel is timed inside the step)",
                "timing": "CUDA events recorded by the library around each kernel, second pass of K steps",
                "in_chain": dom.get("in_chain"),
                "in_chain_timing": "device timestamps inside the undisturbed programmatic-launch chain: return of the "
                                   "kernel's wait on its predecessor -> exit of its last CTA"}

    # ---- CPU baseline: the oracle as it stands, bounded sample
    cpu = None if args.no_cpu_baseline else cpu_baseline(shape, xa_np, xb_np, layers[0], mode, budget_s=12.0)

    tokens_per_s = distrib.whole_job_rate(T, world, ms_per_step)
    out = {
        "metric": "tokens_per_s_through_one_dare_layer", "value": round(tokens_per_s, 1), "unit": "tokens/s",
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 5),
        "us_per_layer": round(ms_per_step * 1e3, 2),
        "timing": {"what": "median over repeats of the K-step region (CUDA events, max over ranks)", "repeats": len(reuse_times),
                   "p10_ms_per_step": round(ms_p10, 5), "p90_ms_per_step": round(ms_p90, 5),
                   "first_region_ms_per_step": round(reuse_times[0], 5), "timed_ms_total": round(sum(reuse_times) * args.steps, 1)},
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(shape, args, n, world),
        "dense": {"ms_per_step": round(dense_ms_per_step, 5), "value": round(world * T / (dense_ms_per_step * 1e-3), 1),
                  "p10_ms_per_step": round(dense_p10, 5), "p90_ms_per_step": round(dense_p90, 5), "repeats": len(dense_times),
                  "clocks": dense_clocks, "first_region_ms_per_step": round(dense_times[0], 5),
                  "speedup_of_reuse_path": round(dense_ms_per_step / ms_per_step, 3)},
        "e2e": {"value": round(world * T / (e2e_ms_per_step * 1e-3), 1), "unit": "tokens/s",
                "ms_per_step": round(e2e_ms_per_step, 5), "p10_ms_per_step": round(e2e_p10, 5),
                "p90_ms_per_step": round(e2e_p90, 5), "repeats": len(long_times), "steps_per_region": long_steps,
                "h2d_bytes_per_step": T * d * 2, "d2h_bytes_per_step": T * d * 2,
                "api": "dare_layer_step_host_async + dare_layer_wait_host (copies overlapped across layer instances); "
                       "wall clock over regions long enough to keep the copy pipeline full",
                "k_step_region_drained": {"ms_per_step": round(e2e_drained_ms, 5), "repeats": len(drained_times),
                                          "what": "the same call over regions of exactly K steps that start and end drained"},
                "synchronous_call": {"api": "dare_layer_step_host", "ms_per_step": round(e2e_sync_ms_per_step, 5),
                                     "value": round(world * T / (e2e_sync_ms_per_step * 1e-3), 1)}},
        "graph_replay": None if graph_ms_per_step is None else
                        {"ms_per_step": round(graph_ms_per_step, 5),
                         "what": "the same steps captured once into a CUDA graph (programmatic launch edges kept) and replayed"},
        "gpu_launches": launches,
        "clocks": clocks,
        "roofline": roofline,
        "kernels": rows,
        "cpu_baseline": cpu,
        "paper_context": "paper reports up to 1.20x per-layer latency reduction (DARE-O, RTX A6000, bf16); not a target",
    }
    print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


def cpu_baseline(shape, xa_np, xb_np, layer0, mode, budget_s):
    """Times the fp64 oracle on the host cores: one dense step to fill its caches, then reuse steps on the same
    A/B buffers until about `budget_s` seconds have gone by."""
    import numpy as np
    from oracle import dare_oracle as orc
    w = {k: layer0._w[k].float().cpu().numpy() for k in ("w_q", "w_k", "w_v", "w_o", "rms_gain")}
    o = orc.OracleLayer(shape.d_model, shape.n_heads, shape.head_dim, shape.batch, shape.seq, shape.rope_theta,
                        shape.rms_eps, w["w_q"], w["w_k"], w["w_v"], w["w_o"], w["rms_gain"])
    o.step(xa_np, mode, TAU)
    bufs = (xb_np, xa_np)
    t0 = time.perf_counter()
    steps = 0
    while True:
        o.step(bufs[steps & 1], mode, TAU)
        steps += 1
        if time.perf_counter() - t0 > budget_s or steps >= 200:
            break
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count()
    return {"value": round(steps * shape.tokens / dt, 1), "unit": "tokens/s", "cores": int(cores), "kind": "oracle",
            "cores_what": "threads of numpy's BLAS pool (threadpoolctl)",
            "sample": f"{steps} reuse steps of the full workload after one dense step, {dt:.1f} s, numpy fp64"}


def run_reference(args):
    """Reference arm: the fp64 oracle on the host cores, same workload, metric and unit."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    from oracle import dare_oracle as orc
    from paper_2605_08134_b200 import workloads as wl
    shape = wl.LLADA_LAYER
    mode = MODES[args.mode]
    w = wl.make_weights(shape)
    hs = wl.HiddenStream(shape, shape.seed)
    xa = hs.first()
    changed = wl.uniform_positions(hs.rng, shape, int(round(args.changed * shape.seq)))
    xb = hs.advance(changed)
    o = orc.OracleLayer(shape.d_model, shape.n_heads, shape.head_dim, shape.batch, shape.seq, shape.rope_theta,
                        shape.rms_eps, w["w_q"], w["w_k"], w["w_v"], w["w_o"], w["rms_gain"])
    o.step(xa, mode, TAU)
    bufs = (xb, xa)
    warm = max(args.warmup, 1)
    steps = min(args.steps, 40)             # bounded sample: each oracle step is a fraction of a second
    for i in range(warm):
        o.step(bufs[i & 1], mode, TAU)
    t0 = time.perf_counter()
    for i in range(steps):
        o.step(bufs[(warm + i) & 1], mode, TAU)
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count()
    value = round(steps * shape.tokens / dt, 1)
    sample = f"{steps} reuse steps of the full workload after one dense step (numpy fp64 oracle)"
    print(json.dumps({
        "impl": "reference", "metric": "tokens_per_s_through_one_dare_layer", "value": value, "unit": "tokens/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": steps, "warmup": warm,
        "ms_per_step": round(dt / steps * 1e3, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": workload_config(shape, args, int(changed.sum()) if mode != 0 else shape.tokens,
                                  int(os.environ.get("WORLD_SIZE", "1"))),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": int(cores), "kind": "oracle",
                         "cores_what": "threads of numpy's BLAS pool (threadpoolctl)", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_micro(args):
    """Memory-bound pieces of the path at a token count large enough to show bandwidth (one JSON line):
    the drift score (Sec. 3.1) and the threshold + compaction (Eq. 2) over 2^24 tokens, head_dim 128."""
    import torch
    from paper_2605_08134_b200 import build
    build.build()
    from paper_2605_08134_b200 import dare
    peaks = load_peaks()
    dev = torch.device("cuda", 0)
    st = torch.cuda.current_stream(dev).cuda_stream
    out = {"metric": "memory_bound_kernels", "unit": "GB/s", "peak": peaks["hbm_gbs"], "peak_source": peaks["source"],
           "kernels": []}

    def time_it(fn, reps=20):
        for _ in range(3):
            fn()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ev0.record()
        for _ in range(reps):
            fn()
        ev1.record()
        torch.cuda.synchronize()
        return ev0.elapsed_time(ev1) / reps * 1e-3

    rows, hd = 1 << 22, 128
    a = torch.randn((rows, hd), device=dev)
    b = a + 0.01 * torch.randn((rows, hd), device=dev)
    sc = torch.empty(rows, device=dev)
    t = time_it(lambda: dare.dare_drift_scores(a.data_ptr(), b.data_ptr(), rows, hd, sc.data_ptr(), st))
    algo = 2.0 * rows * hd * 4 + rows * 4
    out["kernels"].append({"kernel": "drift_scores", "rows": rows, "head_dim": hd, "us": round(t * 1e6, 1),
                           "achieved": round(algo / t / 1e9, 1), "frac": round(algo / t / 1e9 / peaks["hbm_gbs"], 3)})
    del a, b
    # RMSNorm over the rows of the long-context step (batch 4 x 4096 rows of 4096 bf16: 134 MB in, 134 MB out), four
    # input/output pairs in rotation
    rows_n, dm = 16384, 4096
    xs = [torch.randn((rows_n, dm), device=dev).to(torch.bfloat16) for _ in range(4)]
    ys = [torch.empty_like(xs[0]) for _ in range(4)]
    gain = torch.ones(dm, device=dev)
    turn_n = [0]

    def norm():
        i = turn_n[0] & 3
        turn_n[0] += 1
        dare.dare_rmsnorm(xs[i].data_ptr(), gain.data_ptr(), ys[i].data_ptr(), rows_n, dm, 1e-5, dare.BF16, st)

    t = time_it(norm)
    algo = 2.0 * rows_n * dm * 2
    out["kernels"].append({"kernel": "rmsnorm", "rows": rows_n, "d_model": dm, "us": round(t * 1e6, 1),
                           "achieved": round(algo / t / 1e9, 1), "frac": round(algo / t / 1e9 / peaks["hbm_gbs"], 3)})
    ref = xs[0].float()
    ref = (ref * torch.rsqrt((ref * ref).mean(dim=1, keepdim=True) + 1e-5)).to(torch.bfloat16)
    dare.dare_rmsnorm(xs[0].data_ptr(), gain.data_ptr(), ys[0].data_ptr(), rows_n, dm, 1e-5, dare.BF16, st)
    torch.cuda.synchronize()
    assert float((ys[0].float() - ref.float()).abs().max()) <= 0.04, "rmsnorm micro-benchmark: wrong result"
    del xs, ys, ref
    n = 1 << 24
    # four score arrays in rotation (256 MB, twice the L2): every call reads its scores from HBM
    bufs = []
    for i in range(4):
        s = torch.rand(n, device=dev)
        bufs.append(torch.where(s < 0.87, s * 1e-5, s))
    idx = torch.empty(n, dtype=torch.int32, device=dev)
    cnt = torch.zeros(1, dtype=torch.int32, device=dev)
    nb = dare.dare_select_compact_scratch_bytes(n)
    scratch = torch.empty(nb, dtype=torch.uint8, device=dev)
    turn = [0]

    def compact():
        s = bufs[turn[0] & 3]
        turn[0] += 1
        dare.dare_select_compact(s.data_ptr(), n, 0.1, idx.data_ptr(), cnt.data_ptr(), scratch.data_ptr(), nb,
                                 torch.cuda.current_stream(dev).cuda_stream)

    t_stream = time_it(compact)
    # the call is three short launches: issued one by one the host sets the pace, so the figure reported is that of
    # the same calls replayed from a CUDA graph (four calls, one per score array); the stream-launched one is kept
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream(dev)
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        for _ in range(4):
            compact()
    t = time_it(graph.replay) / 4
    k = int(cnt.item())
    algo = 4.0 * n + 4.0 * k            # scores in, index list out
    out["kernels"].append({"kernel": "select_compact", "tokens": n, "refreshed": k, "us": round(t * 1e6, 1),
                           "achieved": round(algo / t / 1e9, 1), "frac": round(algo / t / 1e9 / peaks["hbm_gbs"], 3),
                           "l2": "four score arrays in rotation (256 MB)",
                           "timing": "four calls per CUDA graph, replayed", "us_stream_launched": round(t_stream * 1e6, 1),
                           "bytes_moved": 4.0 * n + 2.0 * (n / 8.0) + 4.0 * k})   # + decision bits out and back in
    print(json.dumps(out))


def run_stack(args):
    """Config 4: the 32-layer LLaDA-8B-shaped stack with random bf16 weights, 256 prompt + 256 generated tokens in
    32-token blocks, one denoising step per generated token, both reuse rules against the dense path.  One JSON line:
    generated tokens per second (wall clock over the whole generation, host loop included)."""
    import numpy as np
    import torch
    from paper_2605_08134_b200 import build
    build.build()
    from paper_2605_08134_b200 import dare, workloads as wl
    shape = wl.LLADA_STACK
    lay = shape.layer
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(shape.seed)
    d, f, V = lay.d_model, shape.d_ff, shape.vocab
    draw = lambda *dims: (torch.randn(dims, generator=gen, device=dev) * 0.02).to(torch.bfloat16)
    ones = torch.ones(d, device=dev)
    w = {"emb": draw(V, d), "head": draw(V, d), "final_gain": ones, "layers": []}
    for _ in range(shape.n_layers):
        w["layers"].append({"w_q": draw(d, d), "w_k": draw(d, d), "w_v": draw(d, d), "w_o": draw(d, d), "rms_gain": ones,
                            "gain2": ones, "w_gate": draw(f, d), "w_up": draw(f, d), "w_down": draw(d, f)})
    B, P = 1, lay.prompt
    stack = dare.Stack(shape, w, B, device=dev)
    prompt = wl.random_prompt(shape, B)
    taus = [TAU] * shape.n_layers
    out = {"metric": "generated_tokens_per_s", "unit": "tokens/s", "data": "synthetic", "dtype": "bf16",
           "config": {"workload": shape.name, "layers": shape.n_layers, "d_model": d, "d_ff": f, "vocab": V,
                      "prompt": P, "generated": shape.gen_len, "block": lay.block, "batch": B, "threshold": TAU}}
    n_gen = min(args.gen, shape.gen_len) if args.gen > 0 else shape.gen_len
    out["config"]["generated"] = n_gen
    final_toks = {}
    for name in ("both", "dense"):
        best = None
        for rep in range(2):
            toks = torch.from_numpy(np.concatenate([prompt, np.full((B, shape.gen_len), shape.mask_id, np.int32)], 1)).to(dev)
            stack.reset()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            refreshed = 0
            for step in range(n_gen):
                stack.decode_step(toks, P, step // lay.block, step == 0, MODES[name], taus)
            torch.cuda.synchronize()
            dt = time.perf_counter() - t0
            best = dt if best is None else min(best, dt)
        assert n_gen < shape.gen_len or not bool((toks == shape.mask_id).any())
        out[name] = {"tokens_per_s": round(n_gen * B / best, 1), "ms_per_token": round(best / n_gen * 1e3, 3)}
        final_toks[name] = toks
    # ---- the same generation with the decode step of every block captured once into a CUDA graph and replayed for
    # the block's tokens (the step takes no decision on the host, so one capture serves a whole block); the first step
    # of the generation (all positions, dense) is enqueued directly.  The host loop never synchronises.
    try:
        best, res = None, tuple(torch.empty(B, dtype=dt_, device=dev) for dt_ in (torch.int32, torch.int32, torch.float32))
        side = torch.cuda.Stream(dev)
        for rep in range(2):
            toks_g = torch.from_numpy(np.concatenate([prompt, np.full((B, shape.gen_len), shape.mask_id, np.int32)], 1)).to(dev)
            stack.reset()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            stack.decode_step_enqueue(toks_g, P, 0, True, MODES["both"], taus, out=res)
            step = 1
            while step < n_gen:
                blk_i = step // lay.block
                n_here = min(n_gen, (blk_i + 1) * lay.block) - step
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    stack.decode_step_enqueue(toks_g, P, blk_i, False, MODES["both"], taus, out=res)
                for _ in range(n_here):
                    graph.replay()
                step += n_here
            torch.cuda.synchronize()
            dt = time.perf_counter() - t0
            best = dt if best is None else min(best, dt)
        assert bool((toks_g == final_toks["both"]).all()), "graph replay generated other tokens than the direct launches"
        out["both_graph"] = {"tokens_per_s": round(n_gen * B / best, 1), "ms_per_token": round(best / n_gen * 1e3, 3),
                             "what": "one CUDA graph per 32-token block, captured inside the timed region"}
    except Exception as e:                # diagnostics only
        print(f"graph replay not measured: {e!r}", file=sys.stderr)
    sel = [stack.layer(l).last_selection(B, lay.seq - P)["count"] for l in range(shape.n_layers)]
    out["value"] = out["both"]["tokens_per_s"]
    out["speedup_of_reuse_path"] = round(out["both"]["tokens_per_s"] / out["dense"]["tokens_per_s"], 3)
    print(json.dumps(out))


def run_sweep(args):
    """Crossover sweep on the long-context layer (batch 4, seq 4096 unless overridden): changed-token fraction
    0..100 % in 5 % steps, uniform and block-clustered patterns, modes kv / o / both against the dense path of the
    same library.  Prints one JSON line with the per-point times and the break-even fraction per mode and pattern
    (running median of three points, then linear interpolation between grid points; null = no crossover below 100 %)."""
    import numpy as np
    import torch
    from paper_2605_08134_b200 import build
    build.build()
    from paper_2605_08134_b200 import dare, workloads as wl
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    base = wl.LLADA_LONG
    shape = wl.scaled(base, batch=args.batch or base.batch, seq=args.seq or base.seq,
                      prompt=(args.seq or base.seq) // 2)
    layers = make_layers(shape, 2, shape.seed, torch, dev, dare)
    gen = torch.Generator(device=dev)
    gen.manual_seed(shape.seed)
    B, S, d = shape.batch, shape.seq, shape.d_model
    xa = torch.randn((B, S, d), generator=gen, device=dev).to(torch.bfloat16)
    y = torch.empty_like(xa)
    rng = np.random.default_rng(shape.seed)
    all_curves = {}

    def changed_mask(frac, pattern):
        n = int(round(frac * S))
        if pattern == "uniform":
            m = wl.uniform_positions(rng, shape, n) if n else np.zeros((B, S), bool)
        else:
            m = wl.clustered_positions(rng, shape, step=4 * 9, clustered_per_seq=n, scattered_per_seq=0)
        return m

    def time_mode(xb, m, steps=args.sweep_steps):
        for lay in layers:
            lay.reset()
            lay.step(xa, m, TAU, y)
        bufs = (xb, xa)
        for i in range(2):
            layers[i % 2].step(bufs[(i // 2) & 1], m, TAU, y)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        ev0.record()
        for i in range(2, 2 + steps):
            layers[i % 2].step(bufs[(i // 2) & 1], m, TAU, y)
        ev1.record()
        torch.cuda.synchronize()
        return ev0.elapsed_time(ev1) / steps * 1e3      # microseconds per layer step

    fracs = [round(0.05 * i, 2) for i in range(21)]
    out = {"metric": "us_per_layer_step_vs_changed_fraction", "config": {"workload": shape.name, "batch": B, "seq_len": S,
           "threshold": TAU, "layers_rotated": 2, "timed_steps_per_point": args.sweep_steps}, "points": [], "break_even": {}}
    # the dense path before, between and after the two patterns (the clocks of these long steps move with the state of
    # the power cap): its median is what the curves are compared with
    dense_runs = [time_mode(xa, 0)]
    for pattern in ("uniform", "clustered"):
        curves = {"kv": [], "o": [], "both": []}
        for f in fracs:
            mask = torch.from_numpy(changed_mask(f, pattern)).to(dev)
            noise = torch.randn((B, S, d), generator=gen, device=dev) * 1e-3
            fresh = torch.randn((B, S, d), generator=gen, device=dev)
            xb = torch.where(mask[:, :, None], fresh, xa.float() + noise).to(torch.bfloat16)
            del noise, fresh
            row = {"pattern": pattern, "changed_fraction": f}
            for name in ("kv", "o", "both"):
                us = time_mode(xb, MODES[name])
                sel = layers[0].last_selection(B, S)
                assert sel["count"] == int(mask.sum().item()), (pattern, f, name, sel["count"])
                row[name + "_us"] = round(us, 1)
                curves[name].append(us)
            out["points"].append(row)
        dense_runs.append(time_mode(xa, 0))
        all_curves[pattern] = curves
    dense_us = statistics.median(dense_runs)
    out["dense_us"] = round(dense_us, 1)
    out["dense_runs_us"] = [round(v, 1) for v in dense_runs]
    worst = 0.0
    for pattern, curves in all_curves.items():
        for name, ys in curves.items():
            worst = max(worst, max(ys) / dense_us)
            be = None
            # a running median of three points first: a single point that met another state of the power cap (they
            # move by +- 3 %, now and then by more) does not decide where the curve crosses the dense path
            ys = [statistics.median(ys[max(0, i - 1):i + 2]) for i in range(len(ys))]
            for i in range(len(fracs) - 1):
                a, b_ = ys[i] - dense_us, ys[i + 1] - dense_us
                if a <= 0 < b_:
                    be = round(fracs[i] + (fracs[i + 1] - fracs[i]) * (-a) / (b_ - a), 3)
                    break
            if be is None and ys[0] > dense_us:
                be = 0.0
            out["break_even"][f"{pattern}/{name}"] = be
    out["worst_ratio_to_dense"] = round(worst, 3)
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mode", default="both", choices=list(MODES))
    ap.add_argument("--changed", type=float, default=0.13)
    ap.add_argument("--layers", type=int, default=8)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-ms", type=float, default=1000.0, help="repeat the K-step region until this much has been timed")
    ap.add_argument("--no-in-chain", action="store_true", help="skip the device-timestamp pass")
    ap.add_argument("--d-model", type=int, default=0, help="exploration: other layer width (multiple of 128)")
    ap.add_argument("--seq", type=int, default=0, help="exploration: other sequence length")
    ap.add_argument("--batch", type=int, default=0, help="exploration: other batch size")
    ap.add_argument("--stack", action="store_true", help="full 32-layer stack generation (config 4) instead")
    ap.add_argument("--gen", type=int, default=0, help="with --stack: stop after this many generated tokens (profiling)")
    ap.add_argument("--sweep", action="store_true", help="long-context crossover sweep (config 5) instead")
    ap.add_argument("--micro", action="store_true", help="time the stand-alone memory-bound kernels instead")
    ap.add_argument("--sweep-steps", type=int, default=20, help="with --sweep: timed steps per point")
    args = ap.parse_args()
    # one process per GPU: under torchrun the world size must be the one asked for; started plainly with --gpus N > 1
    # this process becomes the launcher of N ranks (replicas, NCCL for the barrier and the max over ranks only)
    world_env = os.environ.get("WORLD_SIZE")
    if world_env is not None and int(world_env) != args.gpus and args.impl == "ours" and not (args.stack or args.sweep or args.micro):
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world_env}: start one rank per GPU")
    if world_env is None and args.gpus > 1 and not (args.stack or args.sweep or args.micro):
        import socket
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    if args.stack:
        run_stack(args)
    elif args.sweep:
        run_sweep(args)
    elif args.micro:
        run_micro(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
