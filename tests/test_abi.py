"""The C-ABI library builds, loads and exports every entry point the header
declares; host-side argument checks answer without touching a GPU."""
import ctypes
import os
import re

import pytest

from paper_2502_16886_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(refree_[a-z_0-9]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_functions()
    assert {"refree_score", "refree_select_budget", "refree_compact", "refree_compress_layer"} <= names
    for name in names:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
        assert name in binding.SIGNATURES, f"{name} has no binding"


def test_status_strings_and_defaults(lib):
    assert binding.status_string(0) == "ok"
    assert len({binding.status_string(c) for c in range(8)}) == 8
    d = binding.default_params()
    assert (d.window, d.sink, d.rank_mode, d.scope, d.keep_window, d.force_full, d.dtype) == (1, 4, 0, 0, 1, 0, 1)
    assert abs(d.threshold - 0.01) < 1e-9


def test_params_struct_matches_header_layout(lib):
    # 12 int32/float fields, then 7 int64
    assert ctypes.sizeof(binding.CParams) == 12 * 4 + 7 * 8


def test_host_side_validation_needs_no_gpu(lib):
    good = binding.Params(1, 4, 2, 64, window=8, kv_tokens=128, k_strides=(0, 64, 8192), v_strides=(0, 64, 8192))
    assert binding.refree_workspace_size(good, 128) > 0
    for field, val, code in [("num_q_heads", 3, 1), ("window", 0, 1), ("threshold", 1.0, 1), ("threshold", -0.1, 1),
                             ("head_dim", 96, 2), ("rank_mode", 5, 1), ("dtype", 9, 1), ("num_seqs", 5000, 2)]:
        bad = binding.Params(**{**good.__dict__, field: val})
        with pytest.raises(binding.RefreeError) as ei:
            binding.refree_workspace_size(bad, 128)
        assert ei.value.code == code
    # null pointers and a missing workspace are caught before any launch
    c = good.c_struct()
    rc = lib.refree_score(ctypes.byref(c), None, None, None, None, 128, None, None, 0, None, None)
    assert rc == 1
    fake = ctypes.c_void_p(4096)
    rc = lib.refree_score(ctypes.byref(c), fake, fake, fake, fake, 128, fake, None, 0, None, None)
    assert rc == 3
    rc = lib.refree_score(ctypes.byref(c), fake, ctypes.c_void_p(4100), fake, fake, 128, fake, fake, 1 << 30, None, None)
    assert rc == 2          # K not 16-byte aligned


def test_host_side_validation_of_the_layer_run_inplace_and_paged_entry_points(lib):
    good = binding.Params(1, 4, 2, 64, window=8, kv_tokens=128, k_strides=(0, 64, 8192), v_strides=(0, 64, 8192))
    assert binding.refree_layers_workspace_size(good, 128) == 2 * binding.refree_workspace_size(good, 128)
    c = good.c_struct()
    fake = ctypes.c_void_p(4096)
    one = (ctypes.c_void_p * 1)(4096)
    null1 = (ctypes.c_void_p * 1)(None)
    big = 1 << 30
    # a run of layers: missing arrays, a null layer pointer, one workspace instead of two, nothing to do
    assert lib.refree_compress_layers(ctypes.byref(c), 1, None, one, one, fake, fake, 128, one, one, 256, one, one,
                                      fake, big, None, None) == binding.ERR_INVALID_ARG
    assert lib.refree_compress_layers(ctypes.byref(c), 1, one, null1, one, fake, fake, 128, one, one, 256, one, one,
                                      fake, big, None, None) == binding.ERR_INVALID_ARG
    assert lib.refree_compress_layers(ctypes.byref(c), 1, one, one, one, fake, fake, 128, one, one, 256, one, one,
                                      fake, binding.refree_workspace_size(good, 128), None, None) == binding.ERR_WORKSPACE
    assert lib.refree_compress_layers(ctypes.byref(c), -1, one, one, one, fake, fake, 128, one, one, 256, one, one,
                                      fake, big, None, None) == binding.ERR_INVALID_ARG
    assert lib.refree_compress_layers(ctypes.byref(c), 0, one, one, one, fake, fake, 128, one, one, 256, one, one,
                                      fake, big, None, None) == binding.REFREE_OK
    # in place: unknown anchor, end anchor with score ranking, score ranking without an index list
    assert lib.refree_compact_inplace(ctypes.byref(c), fake, fake, fake, fake, fake, None, 2, None, None) == binding.ERR_INVALID_ARG
    assert lib.refree_compact_inplace(ctypes.byref(c), fake, None, fake, fake, fake, None, 0, None, None) == binding.ERR_INVALID_ARG
    sc = binding.Params(**{**good.__dict__, "rank_mode": binding.RANK_SCORE}).c_struct()
    assert lib.refree_compact_inplace(ctypes.byref(sc), fake, fake, fake, fake, fake, fake, binding.ANCHOR_BACK, None,
                                      None) == binding.ERR_UNSUPPORTED
    assert lib.refree_compact_inplace(ctypes.byref(sc), fake, fake, fake, fake, fake, None, binding.ANCHOR_FRONT, None,
                                      None) == binding.ERR_INVALID_ARG
    assert lib.refree_compress_layer_inplace(ctypes.byref(sc), fake, fake, fake, fake, fake, 128, fake, fake,
                                             binding.ANCHOR_BACK, fake, big, None, None) == binding.ERR_UNSUPPORTED
    assert lib.refree_compress_layer_inplace(ctypes.byref(c), fake, fake, fake, fake, fake, 128, fake, fake,
                                             binding.ANCHOR_BACK, None, 0, None, None) == binding.ERR_WORKSPACE
    # decode over the in-place cache: token-major rows are not back to back
    tm = binding.Params(1, 4, 2, 64, window=8, kv_tokens=128, k_strides=(0, 128, 64), v_strides=(0, 128, 64)).c_struct()
    assert lib.refree_decode_attention_inplace(ctypes.byref(tm), fake, fake, fake, fake, fake, fake, binding.ANCHOR_BACK,
                                               128, fake, fake, big, None, None) == binding.ERR_UNSUPPORTED
    assert lib.refree_decode_attention_inplace(ctypes.byref(c), fake, fake, fake, fake, fake, None, binding.ANCHOR_BACK,
                                               128, fake, fake, big, None, None) == binding.ERR_INVALID_ARG
    assert lib.refree_decode_attention_inplace(ctypes.byref(c), fake, fake, fake, fake, fake, fake, binding.ANCHOR_BACK,
                                               128, fake, None, 0, None, None) == binding.ERR_WORKSPACE
    # paged: block geometry, missing table, unaligned pool, score ranking without offsets
    assert lib.refree_compact_paged(ctypes.byref(c), fake, fake, fake, fake, fake, None, None, fake, 4, 0, fake, fake, 8,
                                    None, None) == binding.ERR_INVALID_ARG
    assert lib.refree_compact_paged(ctypes.byref(c), fake, fake, fake, fake, fake, None, None, None, 4, 16, fake, fake, 8,
                                    None, None) == binding.ERR_INVALID_ARG
    assert lib.refree_compact_paged(ctypes.byref(c), fake, fake, fake, fake, fake, None, None, fake, 4, 16,
                                    ctypes.c_void_p(4100), fake, 8, None, None) == binding.ERR_UNSUPPORTED
    assert lib.refree_compact_paged(ctypes.byref(sc), fake, fake, fake, fake, fake, None, fake, fake, 4, 16, fake, fake, 8,
                                    None, None) == binding.ERR_INVALID_ARG


def test_missing_library_is_an_error(monkeypatch, lib):
    monkeypatch.setattr(binding, "_LIB", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/librefreekv.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.lib()
