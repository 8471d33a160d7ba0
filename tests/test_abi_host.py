"""Host-side checks of the C ABI that need no GPU: the shared library loads, exports every
function include/actqkv.h declares, mirrors the config struct, and rejects bad arguments
before anything is enqueued."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import actqkv_oracle as orc
from paper_2502_13542_b200 import build as lib_build
from paper_2502_13542_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "actqkv.h")


@pytest.fixture(scope="module")
def B():
    lib_build.build()
    from paper_2502_13542_b200 import binding
    return binding


def declared_functions():
    with open(HEADER) as f:
        text = f.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(actqkv_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(B):
    names = declared_functions()
    assert {"actqkv_activation_bias", "actqkv_probe_query", "actqkv_score_blocks", "actqkv_select_cutoff",
            "actqkv_retrieval_attention", "actqkv_append_window"} <= set(names)
    lib = C.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in actqkv.h but not exported"
    # and the binding marshals every one of them
    assert set(names) == set(B.EXPORTED)


def test_config_struct_mirrors_the_header(B):
    with open(HEADER) as f:
        text = f.read()
    body = re.search(r"typedef struct actqkv_config \{(.*?)\} actqkv_config;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = re.findall(r"\b(int32_t|float)\s+([a-z0-9_]+)\s*;", body)
    mirror = [(n, "float" if t is C.c_float else "int32_t") for n, t in B.Config._fields_]
    assert [(n, t) for t, n in fields] == mirror
    assert C.sizeof(B.Config) == 4 * len(fields)


def test_version_and_error_strings(B):
    assert B.version() == 100
    assert B.strerror(0) == "ok"
    seen = {B.strerror(-i) for i in range(1, 7)}
    assert len(seen) == 6 and "unknown actqkv status" not in seen
    assert B.strerror(-99) == "unknown actqkv status"


@pytest.mark.parametrize("spec", [wl.tiny_pr1(), wl.llama3_8b_layer(), wl.decode_batch16(), wl.paper_shaped()])
def test_candidate_count_agrees_with_the_oracle_geometry(B, spec):
    cfg = B.make_config(spec)
    for p0 in list(range(0, 3 * spec.block + spec.n_init + spec.n_local_prev + 5, 7)) + [spec.context - spec.window,
                                                                                        spec.context]:
        init_len, n, _ = orc.key_layout(p0, spec.n_init, spec.block, spec.n_local_prev)
        assert B.n_candidates(cfg, p0) == n, p0


def test_budget_state_size(B):
    cfg = B.make_config(wl.llama3_8b_stack32())
    assert B.budget_state_bytes(cfg) == 8 * (1 + 2 * 32)


def test_bad_arguments_are_rejected_on_the_host(B):
    """NULL / misaligned pointers and unsupported shapes return a negative code before any
    CUDA call is made, so this runs without a device."""
    lib = C.CDLL(B.LIB_PATH)
    cfg = B.make_config(wl.tiny_pr1())
    buf = np.zeros(1 << 16, np.uint8)
    p = buf.ctypes.data
    p += (-p) % 16
    lib.actqkv_activation_bias.restype = C.c_int
    args = [C.c_void_p] * 3 + [C.c_int32] + [C.c_void_p] * 7
    lib.actqkv_activation_bias.argtypes = args
    call = lib.actqkv_activation_bias
    assert call(None, None, p, 256, p, p, p, p, None, None, None) == -1            # NULL config
    assert call(C.byref(cfg), None, None, 256, p, p, p, p, None, None, None) == -1  # NULL q
    assert call(C.byref(cfg), None, p + 4, 256, p, p, p, p, None, None, None) == -2  # misaligned q
    assert call(C.byref(cfg), None, p, 257, p, p, p, p, None, None, None) == -3     # n_tokens > window
    bad = B.make_config(wl.tiny_pr1())
    bad.head_dim = 96
    assert call(C.byref(bad), None, p, 256, p, p, p, p, None, None, None) == -3
    bad = B.make_config(wl.tiny_pr1())
    bad.dtype = 7
    assert call(C.byref(bad), None, p, 256, p, p, p, p, None, None, None) == -4
    batch = B.Batch(1, 2, 0)                                                        # 2 layers of a 1-layer model
    assert call(C.byref(cfg), C.byref(batch), p, 256, p, p, p, p, None, None, None) == -3
