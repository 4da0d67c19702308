"""No-GPU checks of the boundary: the library loads, exports every declared symbol, and validates on the host."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def dare():
    from paper_2605_08134_b200 import build
    build.build()
    from paper_2605_08134_b200 import dare as d
    return d


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(dare_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(dare):
    lib = C.CDLL(dare.LIB_PATH)
    decl = declared_symbols()
    assert len(decl) >= 15
    for name in decl:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    # and the binding wraps each of them under the same name
    for name in decl:
        assert name in dare.EXPORTS, f"binding has no signature for {name}"


def test_status_strings_and_version(dare):
    assert dare.abi_version() >= 1
    seen = {dare.status_string(i) for i in range(10)}
    assert len(seen) == 10 and "ok" in seen
    assert dare.status_string(99) == "unknown status"


def test_workspace_bytes_validates_config(dare):
    good = dare.make_config(256, 4, 64, 1, 128, 1e4, 1e-5, dare.F32)
    n = dare.dare_layer_workspace_bytes(good)
    assert n > 0 and n % 256 == 0
    # grows with the token capacity
    assert dare.dare_layer_workspace_bytes(dare.make_config(256, 4, 64, 2, 128, 1e4, 1e-5, dare.F32)) > n
    bad = [
        dare.make_config(256, 4, 60, 1, 128, 1e4, 1e-5, dare.F32),      # heads * head_dim != d_model
        dare.make_config(256, 4, 64, 0, 128, 1e4, 1e-5, dare.F32),      # no batch
        dare.make_config(256, 4, 64, 1, 128, 1e4, 1e-5, 7),             # unknown dtype
        dare.make_config(256, 4, 64, 1, 128, -1.0, 1e-5, dare.F32),     # theta
        dare.make_config(256, 4, 64, 1, 128, 1e4, 1e-5, dare.F32, score_head=4),
        dare.make_config(192, 4, 48, 1, 128, 1e4, 1e-5, dare.F32),      # head_dim without kernels
    ]
    for cfg in bad:
        assert dare.dare_layer_workspace_bytes(cfg) == 0
    wrong_size = dare.make_config(256, 4, 64, 1, 128, 1e4, 1e-5, dare.F32)
    wrong_size.struct_size = 8
    assert dare.dare_layer_workspace_bytes(wrong_size) == 0
    # the tensor-core path only exists for bf16 with head_dim 128
    assert dare.dare_layer_workspace_bytes(
        dare.make_config(256, 4, 64, 1, 128, 1e4, 1e-5, dare.F32, kernel_path=dare.PATH_TENSOR)) == 0


def test_create_rejects_bad_arguments_before_touching_the_device(dare):
    cfg = dare.make_config(256, 4, 64, 1, 128, 1e4, 1e-5, dare.F32)
    w = dare.LayerWeights(0x1000, 0x2000, 0x3000, 0x4000, 0x5000)
    st, h = dare.dare_layer_create(None, w, 0x10000, 1 << 30)
    assert st == dare.ERR_INVALID_ARG and h is None
    st, h = dare.dare_layer_create(cfg, None, 0x10000, 1 << 30)
    assert st == dare.ERR_INVALID_ARG
    st, h = dare.dare_layer_create(cfg, w, 0, 1 << 30)
    assert st == dare.ERR_INVALID_ARG
    st, h = dare.dare_layer_create(cfg, dare.LayerWeights(0, 0x2000, 0x3000, 0x4000, 0x5000), 0x10000, 1 << 30)
    assert st == dare.ERR_INVALID_ARG
    st, h = dare.dare_layer_create(cfg, dare.LayerWeights(0x1008, 0x2000, 0x3000, 0x4000, 0x5000), 0x10000, 1 << 30)
    assert st == dare.ERR_ALIGN
    st, h = dare.dare_layer_create(cfg, w, 0x10010, 1 << 30)
    assert st == dare.ERR_ALIGN
    st, h = dare.dare_layer_create(cfg, w, 0x10000, 1024)
    assert st == dare.ERR_WORKSPACE
    bad = dare.make_config(192, 4, 48, 1, 128, 1e4, 1e-5, dare.F32)
    st, h = dare.dare_layer_create(bad, w, 0x10000, 1 << 30)
    assert st == dare.ERR_UNSUPPORTED


def test_calls_on_a_null_handle(dare):
    assert dare.dare_layer_step(None, 0x1000, 1, 1, 0, 0, 0.1, 0x2000) == dare.ERR_INVALID_ARG
    assert dare.dare_layer_reset(None) == dare.ERR_INVALID_ARG
    assert dare.dare_layer_destroy(None) == dare.ERR_INVALID_ARG
    assert dare.dare_layer_status(None) == dare.ERR_INVALID_ARG
    assert dare.dare_layer_state_bytes(None) == 0
    assert dare.dare_layer_last_launch_count(None) == 0
