"""ctypes binding of libdare: the same entry points as include/dare.h, argument marshalling only.

Every step of the path runs inside the CUDA library; torch is used by callers for device memory and streams.
Importing this module loads the shared library and fails loudly if it is missing (there is no fallback).
"""
from __future__ import annotations

import ctypes as C
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdare.so")

OK = 0
ERR_INVALID_ARG, ERR_SHAPE, ERR_STATE, ERR_ALIGN, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_UNSUPPORTED, \
    ERR_DEVICE_CHECK = range(1, 10)
MODE_DENSE, MODE_KV, MODE_O, MODE_BOTH = 0, 1, 2, 3
F32, BF16 = 0, 1
PATH_AUTO, PATH_SIMT, PATH_TENSOR = 0, 1, 2


class LayerConfig(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("d_model", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
                ("max_batch", C.c_int32), ("max_seq", C.c_int32), ("rope_theta", C.c_float), ("rms_eps", C.c_float),
                ("dtype", C.c_int32), ("score_head", C.c_int32), ("kernel_path", C.c_int32)]


class LayerWeights(C.Structure):
    _fields_ = [("w_q", C.c_void_p), ("w_k", C.c_void_p), ("w_v", C.c_void_p), ("w_o", C.c_void_p),
                ("rms_gain", C.c_void_p)]


class StackConfig(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_layers", C.c_int32), ("d_ff", C.c_int32), ("vocab", C.c_int32),
                ("mask_id", C.c_int32), ("block", C.c_int32), ("layer", LayerConfig)]


class BlockWeights(C.Structure):
    _fields_ = [("attn", LayerWeights), ("gain2", C.c_void_p), ("w_gate", C.c_void_p), ("w_up", C.c_void_p),
                ("w_down", C.c_void_p)]


class StackWeights(C.Structure):
    _fields_ = [("emb", C.c_void_p), ("head", C.c_void_p), ("final_gain", C.c_void_p),
                ("blocks_host", C.POINTER(BlockWeights))]


class DareError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2605_08134_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, f32, sz = C.c_void_p, C.c_int, C.c_float, C.c_size_t
    sig = {
        "dare_abi_version": (C.c_int, []),
        "dare_status_string": (C.c_char_p, [C.c_int]),
        "dare_layer_workspace_bytes": (sz, [C.POINTER(LayerConfig)]),
        "dare_layer_create": (C.c_int, [C.POINTER(LayerConfig), C.POINTER(LayerWeights), vp, sz, C.POINTER(vp)]),
        "dare_layer_step": (C.c_int, [vp, vp, i32, i32, i32, i32, f32, vp, vp]),
        "dare_layer_step_host": (C.c_int, [vp, vp, i32, i32, i32, i32, f32, vp, vp]),
        "dare_layer_step_host_async": (C.c_int, [vp, vp, i32, i32, i32, i32, f32, vp, vp]),
        "dare_layer_wait_host": (C.c_int, [vp]),
        "dare_layer_step_quantile": (C.c_int, [vp, vp, i32, i32, i32, i32, i32, vp, vp]),
        "dare_layer_last_threshold": (C.c_int, [vp, C.POINTER(C.c_float), vp]),
        "dare_score_kth": (C.c_int, [vp, C.c_int64, C.c_int64, vp, vp]),
        "dare_rmsnorm": (C.c_int, [vp, vp, vp, C.c_int64, i32, f32, i32, vp]),
        "dare_layer_reset": (C.c_int, [vp]),
        "dare_layer_destroy": (C.c_int, [vp]),
        "dare_layer_status": (C.c_int, [vp, vp]),
        "dare_layer_clear_status": (C.c_int, [vp, vp]),
        "dare_layer_debug_wait_probe": (C.c_int, [vp, C.c_uint64, C.POINTER(C.c_uint64), vp]),
        "dare_layer_debug_inject": (C.c_int, [vp, C.c_int]),
        "dare_layer_last_selection": (C.c_int, [vp, vp, vp, vp, vp, vp, vp]),
        "dare_layer_read_caches": (C.c_int, [vp, vp, vp, vp, vp, vp]),
        "dare_layer_state_bytes": (sz, [vp]),
        "dare_layer_export_state": (C.c_int, [vp, vp, sz, vp]),
        "dare_layer_import_state": (C.c_int, [vp, vp, sz, vp]),
        "dare_layer_last_launch_count": (C.c_int, [vp]),
        "dare_layer_set_profiling": (C.c_int, [vp, i32]),
        "dare_layer_last_kernel_times": (C.c_int, [vp, vp, vp, i32, C.POINTER(C.c_int)]),
        "dare_kernel_slot_name": (C.c_char_p, [C.c_int]),
        "dare_stack_workspace_bytes": (sz, [C.POINTER(StackConfig)]),
        "dare_stack_create": (C.c_int, [C.POINTER(StackConfig), C.POINTER(StackWeights), vp, sz, C.POINTER(vp)]),
        "dare_stack_reset": (C.c_int, [vp]),
        "dare_stack_destroy": (C.c_int, [vp]),
        "dare_stack_layer": (vp, [vp, i32]),
        "dare_stack_forward": (C.c_int, [vp, vp, i32, i32, i32, i32, i32, vp, vp, vp]),
        "dare_stack_set_capture": (C.c_int, [vp, i32, vp, vp]),
        "dare_stack_last_hidden": (C.c_int, [vp, vp, sz, vp]),
        "dare_stack_decode_step": (C.c_int, [vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]),
        "dare_layer_debug_timestamps": (C.c_int, [vp, i32, vp, vp]),
        "dare_drift_scores": (C.c_int, [vp, vp, C.c_int64, i32, vp, vp]),
        "dare_select_compact_scratch_bytes": (sz, [C.c_int64]),
        "dare_select_compact": (C.c_int, [vp, C.c_int64, f32, vp, vp, vp, sz, vp]),
        "dare_select_compact_static_max_tokens": (C.c_int64, []),
        "dare_select_compact_static": (C.c_int, [vp, C.c_int64, f32, vp, vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib, tuple(sig)


_lib, EXPORTS = _load()


def status_string(status: int) -> str:
    return _lib.dare_status_string(status).decode()


def abi_version() -> int:
    return _lib.dare_abi_version()


def make_config(d_model, n_heads, head_dim, max_batch, max_seq, rope_theta, rms_eps, dtype, score_head=0,
                kernel_path=PATH_AUTO) -> LayerConfig:
    return LayerConfig(C.sizeof(LayerConfig), d_model, n_heads, head_dim, max_batch, max_seq, rope_theta, rms_eps,
                       dtype, score_head, kernel_path)


def dare_layer_workspace_bytes(cfg: LayerConfig) -> int:
    return _lib.dare_layer_workspace_bytes(C.byref(cfg))


def dare_layer_create(cfg: LayerConfig, weights: LayerWeights, workspace_ptr: int, workspace_bytes: int):
    """-> (status, handle)"""
    out = C.c_void_p()
    st = _lib.dare_layer_create(C.byref(cfg) if cfg is not None else None,
                                C.byref(weights) if weights is not None else None,
                                workspace_ptr, workspace_bytes, C.byref(out))
    return st, out.value


def dare_layer_step(handle, x_ptr, batch, seq_act, pos_begin, mode, threshold, y_ptr, stream=0) -> int:
    return _lib.dare_layer_step(handle, x_ptr, batch, seq_act, pos_begin, mode, threshold, y_ptr, stream)


def dare_layer_step_host(handle, x_host_ptr, batch, seq_act, pos_begin, mode, threshold, y_host_ptr, stream=0) -> int:
    return _lib.dare_layer_step_host(handle, x_host_ptr, batch, seq_act, pos_begin, mode, threshold, y_host_ptr, stream)


def dare_layer_step_host_async(handle, x_host_ptr, batch, seq_act, pos_begin, mode, threshold, y_host_ptr, stream=0) -> int:
    return _lib.dare_layer_step_host_async(handle, x_host_ptr, batch, seq_act, pos_begin, mode, threshold, y_host_ptr,
                                           stream)


def dare_layer_wait_host(handle) -> int:
    return _lib.dare_layer_wait_host(handle)


def dare_layer_reset(handle) -> int:
    return _lib.dare_layer_reset(handle)


def dare_layer_destroy(handle) -> int:
    return _lib.dare_layer_destroy(handle)


def dare_layer_status(handle, stream=0) -> int:
    return _lib.dare_layer_status(handle, stream)


def dare_layer_step_quantile(handle, x_ptr, batch, seq_act, pos_begin, mode, reuse_count, y_ptr, stream=0) -> int:
    return _lib.dare_layer_step_quantile(handle, x_ptr, batch, seq_act, pos_begin, mode, reuse_count, y_ptr, stream)


def dare_layer_last_threshold(handle, stream=0):
    """-> (status, tau of the last step)."""
    tau = C.c_float(0.0)
    st = _lib.dare_layer_last_threshold(handle, C.byref(tau), stream)
    return st, float(tau.value)


def dare_rmsnorm(x_ptr, gain_ptr, y_ptr, rows, d_model, eps, dtype, stream=0) -> int:
    return _lib.dare_rmsnorm(x_ptr, gain_ptr, y_ptr, rows, d_model, eps, dtype, stream)


def dare_score_kth(scores_ptr, n_tokens, k, tau_out_ptr, stream=0) -> int:
    return _lib.dare_score_kth(scores_ptr, n_tokens, k, tau_out_ptr, stream)


def dare_layer_clear_status(handle, stream=0) -> int:
    return _lib.dare_layer_clear_status(handle, stream)


def dare_layer_debug_wait_probe(handle, limit_ns, stream=0):
    """-> (status, nanoseconds the probe's wait took before it gave up)."""
    waited = C.c_uint64(0)
    st = _lib.dare_layer_debug_wait_probe(handle, limit_ns, C.byref(waited), stream)
    return st, int(waited.value)


def dare_layer_debug_inject(handle, what) -> int:
    return _lib.dare_layer_debug_inject(handle, what)


def dare_layer_last_selection(handle, idx_ptr, count_ptr, batch_off_ptr, scores_ptr, delta_ptr, stream=0) -> int:
    return _lib.dare_layer_last_selection(handle, idx_ptr, count_ptr, batch_off_ptr, scores_ptr, delta_ptr, stream)


def dare_layer_read_caches(handle, k_ptr, v_ptr, o_ptr, q_prev_ptr, stream=0) -> int:
    return _lib.dare_layer_read_caches(handle, k_ptr, v_ptr, o_ptr, q_prev_ptr, stream)


def dare_layer_state_bytes(handle) -> int:
    return _lib.dare_layer_state_bytes(handle)


def dare_layer_export_state(handle, dst_ptr, nbytes, stream=0) -> int:
    return _lib.dare_layer_export_state(handle, dst_ptr, nbytes, stream)


def dare_layer_import_state(handle, src_ptr, nbytes, stream=0) -> int:
    return _lib.dare_layer_import_state(handle, src_ptr, nbytes, stream)


def dare_layer_last_launch_count(handle) -> int:
    return _lib.dare_layer_last_launch_count(handle)


def dare_layer_set_profiling(handle, enable: int) -> int:
    return _lib.dare_layer_set_profiling(handle, enable)


def dare_layer_last_kernel_times(handle, slot_ptr, ms_ptr, capacity):
    """-> (status, n)"""
    n = C.c_int(0)
    st = _lib.dare_layer_last_kernel_times(handle, slot_ptr, ms_ptr, capacity, C.byref(n))
    return st, n.value


def dare_layer_debug_timestamps(handle, enable, out_ptr, stream=0) -> int:
    return _lib.dare_layer_debug_timestamps(handle, enable, out_ptr, stream)


def dare_drift_scores(q_now_ptr, q_prev_ptr, rows, head_dim, scores_ptr, stream=0) -> int:
    return _lib.dare_drift_scores(q_now_ptr, q_prev_ptr, rows, head_dim, scores_ptr, stream)


def dare_select_compact_scratch_bytes(n_tokens: int) -> int:
    return _lib.dare_select_compact_scratch_bytes(n_tokens)


def dare_select_compact(scores_ptr, n_tokens, threshold, idx_ptr, count_ptr, scratch_ptr, scratch_bytes, stream=0) -> int:
    return _lib.dare_select_compact(scores_ptr, n_tokens, threshold, idx_ptr, count_ptr, scratch_ptr, scratch_bytes,
                                    stream)


def dare_select_compact_static_max_tokens() -> int:
    return _lib.dare_select_compact_static_max_tokens()


def dare_select_compact_static(scores_ptr, n_tokens, threshold, idx_ptr, count_ptr, stream=0) -> int:
    """dare_select_compact without a scratch argument: for callers that may not allocate device memory."""
    return _lib.dare_select_compact_static(scores_ptr, n_tokens, threshold, idx_ptr, count_ptr, stream)


def dare_kernel_slot_name(slot: int) -> str:
    return _lib.dare_kernel_slot_name(slot).decode()


def dare_stack_workspace_bytes(cfg: StackConfig) -> int:
    return _lib.dare_stack_workspace_bytes(C.byref(cfg))


def dare_stack_create(cfg: StackConfig, weights: StackWeights, workspace_ptr: int, workspace_bytes: int):
    """-> (status, handle)"""
    out = C.c_void_p()
    st = _lib.dare_stack_create(C.byref(cfg), C.byref(weights), workspace_ptr, workspace_bytes, C.byref(out))
    return st, out.value


def dare_stack_reset(handle) -> int:
    return _lib.dare_stack_reset(handle)


def dare_stack_destroy(handle) -> int:
    return _lib.dare_stack_destroy(handle)


def dare_stack_layer(handle, index: int):
    return _lib.dare_stack_layer(handle, index)


def dare_stack_forward(handle, tokens_ptr, batch, seq_total, seq_act, pos_begin, mode, taus_host_ptr, hidden_ptr,
                       stream=0) -> int:
    return _lib.dare_stack_forward(handle, tokens_ptr, batch, seq_total, seq_act, pos_begin, mode, taus_host_ptr,
                                   hidden_ptr, stream)


def dare_stack_set_capture(handle, layer_index, x_ptr, h_ptr) -> int:
    return _lib.dare_stack_set_capture(handle, layer_index, x_ptr, h_ptr)


def dare_stack_last_hidden(handle, dst_host_ptr, nbytes, stream=0) -> int:
    return _lib.dare_stack_last_hidden(handle, dst_host_ptr, nbytes, stream)


def dare_stack_decode_step(handle, tokens_ptr, batch, seq_total, prompt_len, block_index, first, mode, taus_host_ptr,
                           forced_pos_host_ptr, forced_tok_host_ptr, pos_out_ptr, tok_out_ptr, prob_out_ptr,
                           stream=0) -> int:
    return _lib.dare_stack_decode_step(handle, tokens_ptr, batch, seq_total, prompt_len, block_index, first, mode,
                                       taus_host_ptr, forced_pos_host_ptr, forced_tok_host_ptr, pos_out_ptr,
                                       tok_out_ptr, prob_out_ptr, stream)


# ---------------------------------------------------------------------------------------------------------------
class Layer:
    """Convenience wrapper: owns the torch tensors behind a handle (weights, workspace) and marshals pointers.

    No arithmetic happens here.  `x`/`y` are torch CUDA tensors (or pinned host tensors for `step_host`).
    """

    def __init__(self, shape, weights: dict, device="cuda:0", kernel_path=PATH_AUTO, max_batch=None, max_seq=None,
                 score_head=0):
        import numpy as np
        import torch
        self.torch = torch
        self.shape = shape
        self.device = torch.device(device)
        self.tdtype = torch.bfloat16 if shape.dtype == BF16 else torch.float32
        self.max_batch = max_batch or shape.batch
        self.max_seq = max_seq or shape.seq
        self.cfg = make_config(shape.d_model, shape.n_heads, shape.head_dim, self.max_batch, self.max_seq,
                               shape.rope_theta, shape.rms_eps, shape.dtype, score_head, kernel_path)
        self._w = {}
        for k in ("w_q", "w_k", "w_v", "w_o"):
            v = weights[k]
            t = v if isinstance(v, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(v, np.float32))
            self._w[k] = t.to(self.device, self.tdtype).contiguous()
        g = weights["rms_gain"]
        g = g if isinstance(g, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(g, np.float32))
        self._w["rms_gain"] = g.to(self.device, torch.float32).contiguous()
        self.wstruct = LayerWeights(*(self._w[k].data_ptr() for k in ("w_q", "w_k", "w_v", "w_o", "rms_gain")))
        nbytes = dare_layer_workspace_bytes(self.cfg)
        if nbytes == 0:
            raise DareError(ERR_UNSUPPORTED, "dare_layer_workspace_bytes")
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        with torch.cuda.device(self.device):
            st, self.handle = dare_layer_create(self.cfg, self.wstruct, base, nbytes)
        if st != OK:
            raise DareError(st, "dare_layer_create")

    def _stream(self):
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def step(self, x, mode, threshold, y=None, pos_begin=0):
        torch = self.torch
        assert x.is_cuda and x.dtype == self.tdtype and x.is_contiguous()
        if y is None:
            y = torch.empty_like(x)
        st = dare_layer_step(self.handle, x.data_ptr(), x.shape[0], x.shape[1], pos_begin, mode, threshold,
                             y.data_ptr(), self._stream())
        if st != OK:
            raise DareError(st, "dare_layer_step")
        return y

    def step_quantile(self, x, mode, reuse_count, y=None, pos_begin=0):
        """The step with the threshold taken from its own scores: the `reuse_count` least-drifted tokens are reused."""
        torch = self.torch
        assert x.is_cuda and x.dtype == self.tdtype and x.is_contiguous()
        if y is None:
            y = torch.empty_like(x)
        st = dare_layer_step_quantile(self.handle, x.data_ptr(), x.shape[0], x.shape[1], pos_begin, mode, reuse_count,
                                      y.data_ptr(), self._stream())
        if st != OK:
            raise DareError(st, "dare_layer_step_quantile")
        return y

    def last_threshold(self) -> float:
        st, tau = dare_layer_last_threshold(self.handle, self._stream())
        if st != OK:
            raise DareError(st, "dare_layer_last_threshold")
        return tau

    def step_host(self, x_host, mode, threshold, y_host, pos_begin=0):
        st = dare_layer_step_host(self.handle, x_host.data_ptr(), x_host.shape[0], x_host.shape[1], pos_begin, mode,
                                  threshold, y_host.data_ptr(), self._stream())
        if st != OK:
            raise DareError(st, "dare_layer_step_host")
        return y_host

    def step_host_async(self, x_host, mode, threshold, y_host, pos_begin=0):
        """Enqueue only: y_host is defined after wait_host(); x_host must stay valid until then."""
        st = dare_layer_step_host_async(self.handle, x_host.data_ptr(), x_host.shape[0], x_host.shape[1], pos_begin, mode,
                                        threshold, y_host.data_ptr(), self._stream())
        if st != OK:
            raise DareError(st, "dare_layer_step_host_async")

    def wait_host(self):
        st = dare_layer_wait_host(self.handle)
        if st != OK:
            raise DareError(st, "dare_layer_wait_host")

    def reset(self):
        st = dare_layer_reset(self.handle)
        if st != OK:
            raise DareError(st, "dare_layer_reset")

    def status(self) -> int:
        return dare_layer_status(self.handle, self._stream())

    def clear_status(self):
        st = dare_layer_clear_status(self.handle, self._stream())
        if st != OK:
            raise DareError(st, "dare_layer_clear_status")

    def wait_probe(self, limit_ns):
        st, waited = dare_layer_debug_wait_probe(self.handle, limit_ns, self._stream())
        if st != OK:
            raise DareError(st, "dare_layer_debug_wait_probe")
        return waited

    def inject(self, what):
        st = dare_layer_debug_inject(self.handle, what)
        if st != OK:
            raise DareError(st, "dare_layer_debug_inject")

    def last_selection(self, batch, seq_act):
        """-> dict(idx, count, batch_off, scores, delta) as numpy arrays."""
        import numpy as np
        T = batch * seq_act
        idx = np.zeros(T, np.int32)
        cnt = np.zeros(1, np.int32)
        boff = np.zeros(batch + 1, np.int32)
        sc = np.zeros(T, np.float32)
        dl = np.zeros(T, np.int32)
        st = dare_layer_last_selection(self.handle, idx.ctypes.data, cnt.ctypes.data, boff.ctypes.data,
                                       sc.ctypes.data, dl.ctypes.data, self._stream())
        if st != OK:
            raise DareError(st, "dare_layer_last_selection")
        n = int(cnt[0])
        return {"idx": idx[:n].copy(), "count": n, "batch_off": boff, "scores": sc, "delta": dl.reshape(batch, seq_act)}

    def read_caches(self, batch, kv_len):
        """-> dict(k, v, o, q_prev) as float32 numpy arrays [batch, kv_len, ...]."""
        import numpy as np
        torch = self.torch
        d, hd = self.shape.d_model, self.shape.head_dim
        host = [torch.empty((batch, kv_len, d), dtype=self.tdtype) for _ in range(3)]
        qp = np.zeros((batch, kv_len, hd), np.float32)
        st = dare_layer_read_caches(self.handle, host[0].data_ptr(), host[1].data_ptr(), host[2].data_ptr(),
                                    qp.ctypes.data, self._stream())
        if st != OK:
            raise DareError(st, "dare_layer_read_caches")
        k, v, o = (h.float().numpy() for h in host)
        return {"k": k, "v": v, "o": o, "q_prev": qp}

    def set_profiling(self, enable: bool):
        st = dare_layer_set_profiling(self.handle, 1 if enable else 0)
        if st != OK:
            raise DareError(st, "dare_layer_set_profiling")

    def kernel_times(self):
        """-> list of (kernel name, milliseconds) of the last step, in launch order (profiling must be on)."""
        import numpy as np
        slots = np.zeros(16, np.int32)
        ms = np.zeros(16, np.float32)
        st, n = dare_layer_last_kernel_times(self.handle, slots.ctypes.data, ms.ctypes.data, 16)
        if st != OK:
            raise DareError(st, "dare_layer_last_kernel_times")
        return [(dare_kernel_slot_name(int(slots[i])), float(ms[i])) for i in range(n)]

    def debug_timestamps(self, enable=True):
        """-> uint64[8, 8] phase timestamps (ns) of the tensor-core kernels of the last step; see include/dare.h."""
        import numpy as np
        out = np.zeros(64 + 3 * 1024, np.uint64)
        st = dare_layer_debug_timestamps(self.handle, 1 if enable else 0, out.ctypes.data, self._stream())
        if st != OK:
            raise DareError(st, "dare_layer_debug_timestamps")
        self.debug_blocks = out[64:].reshape(1024, 3)
        return out[:64].reshape(8, 8)

    def launch_count(self) -> int:
        return dare_layer_last_launch_count(self.handle)

    def close(self):
        if getattr(self, "handle", None):
            dare_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class _LayerView(Layer):
    """A layer that belongs to a stack: same observation calls, no ownership."""

    def __init__(self, handle, shape, torch, device):
        self.handle, self.shape, self.torch, self.device = handle, shape, torch, device
        self.tdtype = torch.bfloat16

    def close(self):
        self.handle = None


class Stack:
    """Convenience wrapper around dare_stack_*: owns the device copies of the weights and the workspace."""

    def __init__(self, sshape, weights: dict, batch: int, device="cuda:0"):
        import numpy as np
        import torch
        self.torch, self.sshape, self.batch = torch, sshape, batch
        self.device = torch.device(device)
        lay = sshape.layer
        dev = lambda a, dt: (a if isinstance(a, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(a, np.float32))) \
            .to(self.device, dt).contiguous()
        bf, f32 = torch.bfloat16, torch.float32
        self._keep = [dev(weights["emb"], bf), dev(weights["head"], bf), dev(weights["final_gain"], f32)]
        blocks = (BlockWeights * sshape.n_layers)()
        for l, lw in enumerate(weights["layers"]):
            t = {k: dev(lw[k], bf) for k in ("w_q", "w_k", "w_v", "w_o", "w_gate", "w_up", "w_down")}
            t["rms_gain"], t["gain2"] = dev(lw["rms_gain"], f32), dev(lw["gain2"], f32)
            self._keep.append(t)
            blocks[l] = BlockWeights(LayerWeights(t["w_q"].data_ptr(), t["w_k"].data_ptr(), t["w_v"].data_ptr(),
                                                  t["w_o"].data_ptr(), t["rms_gain"].data_ptr()),
                                     t["gain2"].data_ptr(), t["w_gate"].data_ptr(), t["w_up"].data_ptr(),
                                     t["w_down"].data_ptr())
        self._blocks = blocks
        lcfg = make_config(lay.d_model, lay.n_heads, lay.head_dim, batch, lay.seq, lay.rope_theta, lay.rms_eps, BF16, 0,
                           PATH_TENSOR)
        self.cfg = StackConfig(C.sizeof(StackConfig), sshape.n_layers, sshape.d_ff, sshape.vocab, sshape.mask_id,
                               lay.block, lcfg)
        self.w = StackWeights(self._keep[0].data_ptr(), self._keep[1].data_ptr(), self._keep[2].data_ptr(), blocks)
        nbytes = dare_stack_workspace_bytes(self.cfg)
        if nbytes == 0:
            raise DareError(ERR_UNSUPPORTED, "dare_stack_workspace_bytes")
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        with torch.cuda.device(self.device):
            st, self.handle = dare_stack_create(self.cfg, self.w, base, nbytes)
        if st != OK:
            raise DareError(st, "dare_stack_create")

    def _stream(self):
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def layer(self, index: int) -> "_LayerView":
        return _LayerView(dare_stack_layer(self.handle, index), self.sshape.layer, self.torch, self.device)

    def reset(self):
        dare_stack_reset(self.handle)

    def forward(self, tokens, seq_act, pos_begin, mode, taus):
        """tokens: int32 CUDA tensor [batch, seq_total]; -> bf16 hidden states [batch, seq_act, d_model]."""
        import numpy as np
        torch = self.torch
        taus = np.ascontiguousarray(taus, np.float32)
        out = torch.empty((tokens.shape[0], seq_act, self.sshape.layer.d_model), dtype=torch.bfloat16, device=self.device)
        st = dare_stack_forward(self.handle, tokens.data_ptr(), tokens.shape[0], tokens.shape[1], seq_act, pos_begin, mode,
                                taus.ctypes.data, out.data_ptr(), self._stream())
        if st != OK:
            raise DareError(st, "dare_stack_forward")
        return out

    def decode_step(self, tokens, prompt_len, block_index, first, mode, taus, forced=None):
        """-> (pos, tok, prob) numpy arrays [batch]: the step's own choice; `tokens` is updated in place."""
        import numpy as np
        torch = self.torch
        B = tokens.shape[0]
        taus = np.ascontiguousarray(taus, np.float32)
        pos = torch.empty(B, dtype=torch.int32, device=self.device)
        tok = torch.empty(B, dtype=torch.int32, device=self.device)
        prob = torch.empty(B, dtype=torch.float32, device=self.device)
        fp = ft = None
        if forced is not None:
            fp = np.ascontiguousarray(forced[0], np.int32)
            ft = np.ascontiguousarray(forced[1], np.int32)
        st = dare_stack_decode_step(self.handle, tokens.data_ptr(), B, tokens.shape[1], prompt_len, block_index,
                                    1 if first else 0, mode, taus.ctypes.data,
                                    fp.ctypes.data if fp is not None else None, ft.ctypes.data if ft is not None else None,
                                    pos.data_ptr(), tok.data_ptr(), prob.data_ptr(), self._stream())
        if st != OK:
            raise DareError(st, "dare_stack_decode_step")
        torch.cuda.synchronize(self.device)       # the forced arrays are host memory read by an async copy
        return pos.cpu().numpy(), tok.cpu().numpy(), prob.cpu().numpy()

    def decode_step_enqueue(self, tokens, prompt_len, block_index, first, mode, taus, out=None):
        """Enqueue-only form of decode_step (no forced choice, no synchronisation, nothing allocated when `out` is
        given): usable inside a CUDA-graph capture.  -> (pos, tok, prob) device tensors [batch]."""
        import numpy as np
        torch = self.torch
        B = tokens.shape[0]
        taus = np.ascontiguousarray(taus, np.float32)
        if out is None:
            out = (torch.empty(B, dtype=torch.int32, device=self.device),
                   torch.empty(B, dtype=torch.int32, device=self.device),
                   torch.empty(B, dtype=torch.float32, device=self.device))
        st = dare_stack_decode_step(self.handle, tokens.data_ptr(), B, tokens.shape[1], prompt_len, block_index,
                                    1 if first else 0, mode, taus.ctypes.data, None, None,
                                    out[0].data_ptr(), out[1].data_ptr(), out[2].data_ptr(), self._stream())
        if st != OK:
            raise DareError(st, "dare_stack_decode_step")
        return out

    def set_capture(self, layer_index, x_buf=None, h_buf=None):
        st = dare_stack_set_capture(self.handle, layer_index, x_buf.data_ptr() if x_buf is not None else None,
                                    h_buf.data_ptr() if h_buf is not None else None)
        if st != OK:
            raise DareError(st, "dare_stack_set_capture")

    def last_hidden(self, batch, seq_act):
        """-> float32 numpy [batch, seq_act, d_model]: final-normed states of the last pass."""
        torch = self.torch
        h = torch.empty((batch, seq_act, self.sshape.layer.d_model), dtype=torch.bfloat16)
        st = dare_stack_last_hidden(self.handle, h.data_ptr(), h.numel() * 2, self._stream())
        if st != OK:
            raise DareError(st, "dare_stack_last_hidden")
        return h.float().numpy()

    def close(self):
        if getattr(self, "handle", None):
            dare_stack_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
