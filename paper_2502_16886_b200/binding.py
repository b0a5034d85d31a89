"""ctypes binding of ``librefreekv.so``: same names as the C ABI, argument
marshalling only.  Every step of the pass runs in the CUDA kernels of the
library; there is no CPU fallback, and a missing library is an error.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
from typing import Optional

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "librefreekv.so")

REFREE_OK = 0
STATUS_NAMES = ["OK", "INVALID_ARG", "UNSUPPORTED", "WORKSPACE", "CAPACITY", "CUDA", "TIMEOUT", "NONFINITE",
                "STATIC_LIMIT"]
(ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CAPACITY, ERR_CUDA, ERR_TIMEOUT, ERR_NONFINITE,
 ERR_STATIC_LIMIT) = range(1, 9)
STATIC_SCRATCH_BYTES = 256 * 1024
DEV_CAPACITY, DEV_TIMEOUT, DEV_NONFINITE = 1, 2, 4
RANK_POSITION, RANK_SCORE = 0, 1
SCOPE_HEAD, SCOPE_LAYER = 0, 1
DTYPE_F32, DTYPE_BF16 = 0, 1
ANCHOR_FRONT, ANCHOR_BACK = 0, 1


class RefreeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        name = STATUS_NAMES[code] if 0 <= code < len(STATUS_NAMES) else str(code)
        super().__init__(f"{where}: REFREE_ERR_{name} ({status_string(code)})")


class CParams(ctypes.Structure):
    _fields_ = [
        ("num_seqs", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("window", ctypes.c_int32), ("sink", ctypes.c_int32),
        ("threshold", ctypes.c_float),
        ("rank_mode", ctypes.c_int32), ("scope", ctypes.c_int32),
        ("keep_window", ctypes.c_int32), ("force_full", ctypes.c_int32),
        ("dtype", ctypes.c_int32),
        ("kv_tokens", ctypes.c_int64),
        ("k_stride_seq", ctypes.c_int64), ("k_stride_tok", ctypes.c_int64), ("k_stride_head", ctypes.c_int64),
        ("v_stride_seq", ctypes.c_int64), ("v_stride_tok", ctypes.c_int64), ("v_stride_head", ctypes.c_int64),
    ]


@dataclasses.dataclass
class Params:
    """Mirror of ``refree_params`` (see ``include/refreekv.h``)."""
    num_seqs: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    window: int = 1
    sink: int = 4
    threshold: float = 0.01
    rank_mode: int = RANK_POSITION
    scope: int = SCOPE_HEAD
    keep_window: int = 1
    force_full: int = 0
    dtype: int = DTYPE_BF16
    kv_tokens: int = 0
    k_strides: tuple = (0, 0, 0)   # (seq, tok, head) in elements
    v_strides: tuple = (0, 0, 0)

    def c_struct(self) -> CParams:
        return CParams(self.num_seqs, self.num_q_heads, self.num_kv_heads, self.head_dim,
                       self.window, self.sink, self.threshold, self.rank_mode, self.scope,
                       self.keep_window, self.force_full, self.dtype, self.kv_tokens,
                       *self.k_strides, *self.v_strides)


_LIB = None
_VP, _I64, _SZ = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
_PP = ctypes.POINTER(CParams)

SIGNATURES = {
    "refree_default_params": (None, [_PP]),
    "refree_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "refree_kernel_launch_count": (ctypes.c_int64, []),
    "refree_workspace_size": (ctypes.c_int, [_PP, _I64, ctypes.POINTER(_SZ)]),
    "refree_score": (ctypes.c_int, [_PP, _VP, _VP, _VP, _VP, _I64, _VP, _VP, _SZ, _VP, _VP]),
    "refree_select_budget": (ctypes.c_int, [_PP, _VP, _VP, _I64, _VP, _VP, _VP, _I64, _VP, _SZ, _VP, _VP]),
    "refree_select_budget_static": (ctypes.c_int, [_PP, _VP, _VP, _I64, _VP, _VP, _VP, _I64, _VP, _VP]),
    "refree_compact": (ctypes.c_int, [_PP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _I64, _VP, _VP]),
    "refree_compact_paged": (ctypes.c_int, [_PP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, _VP, ctypes.c_int32, ctypes.c_int32,
                                            _VP, _VP, _I64, _VP, _VP]),
    "refree_compact_inplace": (ctypes.c_int, [_PP, _VP, _VP, _VP, _VP, _VP, _VP, ctypes.c_int32, _VP, _VP]),
    "refree_compress_layer_inplace": (ctypes.c_int, [_PP, _VP, _VP, _VP, _VP, _VP, _I64, _VP, _VP, ctypes.c_int32, _VP, _SZ,
                                                     _VP, _VP]),
    "refree_compress_layer": (ctypes.c_int, [_PP, _VP, _VP, _VP, _VP, _VP, _I64, _VP, _VP, _I64, _VP, _VP,
                                             _VP, _VP, _VP, _SZ, _VP, _VP]),
    "refree_layers_workspace_size": (ctypes.c_int, [_PP, _I64, ctypes.POINTER(_SZ)]),
    "refree_compress_layers": (ctypes.c_int, [_PP, ctypes.c_int32, _VP, _VP, _VP, _VP, _VP, _I64, _VP, _VP, _I64,
                                              _VP, _VP, _VP, _SZ, _VP, _VP]),
    "refree_host_pipeline_arena_size": (ctypes.c_int, [_PP, _I64, _I64, _I64, ctypes.POINTER(_SZ)]),
    "refree_compress_layers_host": (ctypes.c_int, [_PP, ctypes.c_int32, _VP, _VP, _VP, _I64, _VP, _VP, _I64, _VP, _VP,
                                                   _I64, _VP, _VP, _VP, _SZ]),
    "refree_decode_workspace_size": (ctypes.c_int, [_PP, _I64, ctypes.POINTER(_SZ)]),
    "refree_decode_attention": (ctypes.c_int, [_PP, _VP, _VP, _VP, _VP, _I64, _VP, _VP, _SZ, _VP, _VP]),
    "refree_decode_attention_inplace": (ctypes.c_int, [_PP, _VP, _VP, _VP, _VP, _VP, _VP, ctypes.c_int32, _I64, _VP, _VP,
                                                       _SZ, _VP, _VP]),
    "refree_sol_read_stream": (ctypes.c_int, [_VP, _I64, _VP, _VP]),
    "refree_sol_row_mix": (ctypes.c_int, [_VP, _VP, _VP, _VP, _I64, _I64, ctypes.c_int32, _VP, _VP]),
    "refree_host_arena_size": (ctypes.c_int, [_PP, _I64, _I64, _I64, ctypes.POINTER(_SZ)]),
    "refree_compress_layer_host": (ctypes.c_int, [_PP, _VP, _VP, _VP, _I64, _VP, _VP, _I64, _VP, _VP, _I64,
                                                  _VP, _VP, _VP, _VP, _VP, _SZ, _VP]),
}


def lib():
    """Load the CUDA library (once).  Raises if it has not been built."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2502_16886_b200.build` "
                "(there is no CPU fallback)")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _LIB = handle
    return _LIB


def status_string(code: int) -> str:
    return lib().refree_status_string(int(code)).decode()


def refree_kernel_launch_count() -> int:
    return int(lib().refree_kernel_launch_count())


def default_params() -> CParams:
    c = CParams()
    lib().refree_default_params(ctypes.byref(c))
    return c


def _dp(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check(code: int, where: str):
    if code != REFREE_OK:
        raise RefreeError(code, where)


def refree_workspace_size(p: Params, total_tokens: int) -> int:
    out = _SZ(0)
    c = p.c_struct()
    _check(lib().refree_workspace_size(ctypes.byref(c), total_tokens, ctypes.byref(out)), "refree_workspace_size")
    return int(out.value)


def refree_score(p: Params, q_win, k, seq_start, seq_len, total_tokens, scores, workspace,
                 device_status=None, stream=None, check=True) -> int:
    c = p.c_struct()
    rc = lib().refree_score(ctypes.byref(c), _dp(q_win), _dp(k), _dp(seq_start), _dp(seq_len), total_tokens,
                            _dp(scores), _dp(workspace), workspace.numel() * workspace.element_size() if workspace is not None else 0,
                            _dp(device_status), _stream(stream))
    if check:
        _check(rc, "refree_score")
    return rc


def refree_select_budget(p: Params, scores, seq_len, total_tokens, lengths, offsets, kept_idx, capacity_rows,
                         workspace, device_status=None, stream=None, check=True) -> int:
    c = p.c_struct()
    rc = lib().refree_select_budget(ctypes.byref(c), _dp(scores), _dp(seq_len), total_tokens, _dp(lengths),
                                    _dp(offsets), _dp(kept_idx), capacity_rows, _dp(workspace),
                                    workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                    _dp(device_status), _stream(stream))
    if check:
        _check(rc, "refree_select_budget")
    return rc


def refree_select_budget_static(p: Params, scores, seq_len, total_tokens, lengths, offsets, kept_idx, capacity_rows,
                                device_status=None, stream=None, check=True) -> int:
    """Selection with the library's built-in scratch: takes no workspace and
    allocates nothing (see the header for who needs this and for its limits)."""
    c = p.c_struct()
    rc = lib().refree_select_budget_static(ctypes.byref(c), _dp(scores), _dp(seq_len), total_tokens, _dp(lengths),
                                           _dp(offsets), _dp(kept_idx), capacity_rows, _dp(device_status),
                                           _stream(stream))
    if check:
        _check(rc, "refree_select_budget_static")
    return rc


def refree_compact(p: Params, k, v, seq_start, seq_len, lengths, offsets, kept_idx, k_out, v_out, capacity_rows,
                   device_status=None, stream=None, check=True) -> int:
    c = p.c_struct()
    rc = lib().refree_compact(ctypes.byref(c), _dp(k), _dp(v), _dp(seq_start), _dp(seq_len), _dp(lengths),
                              _dp(offsets), _dp(kept_idx), _dp(k_out), _dp(v_out), capacity_rows,
                              _dp(device_status), _stream(stream))
    if check:
        _check(rc, "refree_compact")
    return rc


def refree_compact_paged(p: Params, k, v, seq_start, seq_len, lengths, offsets, kept_idx, block_table, block_rows,
                         k_pool, v_pool, device_status=None, stream=None, check=True) -> int:
    """``block_table`` is int32 ``[units, max_blocks_per_unit]``; the pools are ``[num_blocks, block_rows, d]``."""
    c = p.c_struct()
    rc = lib().refree_compact_paged(ctypes.byref(c), _dp(k), _dp(v), _dp(seq_start), _dp(seq_len), _dp(lengths),
                                    _dp(offsets), _dp(kept_idx), _dp(block_table), block_table.shape[1], block_rows,
                                    _dp(k_pool), _dp(v_pool), k_pool.shape[0], _dp(device_status), _stream(stream))
    if check:
        _check(rc, "refree_compact_paged")
    return rc


def refree_compact_inplace(p: Params, k, v, seq_start, seq_len, offsets, kept_idx, device_status=None, stream=None,
                           check=True, anchor=ANCHOR_FRONT) -> int:
    """Gathers every unit's kept rows at the front (or, ``ANCHOR_BACK``, the end) of its own region of ``k`` and ``v``."""
    c = p.c_struct()
    rc = lib().refree_compact_inplace(ctypes.byref(c), _dp(k), _dp(v), _dp(seq_start), _dp(seq_len), _dp(offsets),
                                      _dp(kept_idx), anchor, _dp(device_status), _stream(stream))
    if check:
        _check(rc, "refree_compact_inplace")
    return rc


def refree_compress_layer_inplace(p: Params, q_win, k, v, seq_start, seq_len, total_tokens, lengths, offsets, anchor,
                                  workspace, device_status=None, stream=None, check=True) -> int:
    c = p.c_struct()
    rc = lib().refree_compress_layer_inplace(ctypes.byref(c), _dp(q_win), _dp(k), _dp(v), _dp(seq_start), _dp(seq_len),
                                             total_tokens, _dp(lengths), _dp(offsets), anchor, _dp(workspace),
                                             workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                             _dp(device_status), _stream(stream))
    if check:
        _check(rc, "refree_compress_layer_inplace")
    return rc


def refree_compress_layer(p: Params, q_win, k, v, seq_start, seq_len, total_tokens, k_out, v_out, capacity_rows,
                          lengths, offsets, kept_idx, scores, workspace, device_status=None, stream=None,
                          check=True) -> int:
    c = p.c_struct()
    rc = lib().refree_compress_layer(ctypes.byref(c), _dp(q_win), _dp(k), _dp(v), _dp(seq_start), _dp(seq_len),
                                     total_tokens, _dp(k_out), _dp(v_out), capacity_rows, _dp(lengths),
                                     _dp(offsets), _dp(kept_idx), _dp(scores), _dp(workspace),
                                     workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                     _dp(device_status), _stream(stream))
    if check:
        _check(rc, "refree_compress_layer")
    return rc


def refree_decode_workspace_size(p: Params, max_rows_per_unit: int) -> int:
    out = _SZ(0)
    c = p.c_struct()
    _check(lib().refree_decode_workspace_size(ctypes.byref(c), max_rows_per_unit, ctypes.byref(out)),
           "refree_decode_workspace_size")
    return int(out.value)


def refree_decode_attention(p: Params, q_new, k_c, v_c, offsets, max_rows_per_unit, out, workspace,
                            device_status=None, stream=None, check=True) -> int:
    c = p.c_struct()
    rc = lib().refree_decode_attention(ctypes.byref(c), _dp(q_new), _dp(k_c), _dp(v_c), _dp(offsets),
                                       max_rows_per_unit, _dp(out), _dp(workspace),
                                       workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                       _dp(device_status), _stream(stream))
    if check:
        _check(rc, "refree_decode_attention")
    return rc


def refree_decode_attention_inplace(p: Params, q_new, k, v, seq_start, seq_len, lengths, anchor, max_rows_per_unit, out,
                                    workspace, device_status=None, stream=None, check=True) -> int:
    c = p.c_struct()
    rc = lib().refree_decode_attention_inplace(ctypes.byref(c), _dp(q_new), _dp(k), _dp(v), _dp(seq_start), _dp(seq_len),
                                               _dp(lengths), anchor, max_rows_per_unit, _dp(out), _dp(workspace),
                                               workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                               _dp(device_status), _stream(stream))
    if check:
        _check(rc, "refree_decode_attention_inplace")
    return rc


def refree_host_arena_size(p: Params, total_tokens: int, kv_elems: int, capacity_rows: int) -> int:
    out = _SZ(0)
    c = p.c_struct()
    _check(lib().refree_host_arena_size(ctypes.byref(c), total_tokens, kv_elems, capacity_rows, ctypes.byref(out)),
           "refree_host_arena_size")
    return int(out.value)


def refree_compress_layer_host(p: Params, q_win, k, v, seq_start, seq_len, total_tokens, k_out, v_out,
                               capacity_rows, lengths, offsets, kept_idx, scores, arena, stream=None,
                               check=True) -> int:
    """All tensors but ``arena`` are CPU tensors (pinned or pageable)."""
    c = p.c_struct()
    rc = lib().refree_compress_layer_host(ctypes.byref(c), _dp(q_win), _dp(k), _dp(v), k.numel(), _dp(seq_start),
                                          _dp(seq_len), total_tokens, _dp(k_out), _dp(v_out), capacity_rows,
                                          _dp(lengths), _dp(offsets), _dp(kept_idx), _dp(scores), _dp(arena),
                                          arena.numel() * arena.element_size(), _stream(stream))
    if check:
        _check(rc, "refree_compress_layer_host")
    return rc


# ---- convenience wrapper -----------------------------------------------------
def refree_host_pipeline_arena_size(p: Params, total_tokens: int, kv_elems: int, capacity_rows: int) -> int:
    out = _SZ(0)
    c = p.c_struct()
    _check(lib().refree_host_pipeline_arena_size(ctypes.byref(c), total_tokens, kv_elems, capacity_rows,
                                                 ctypes.byref(out)), "refree_host_pipeline_arena_size")
    return int(out.value)


def _ptr_array(tensors):
    arr = (ctypes.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = t.data_ptr()
    return arr


def refree_compress_layers_host(p: Params, q_win, k, v, seq_start, seq_len, total_tokens, k_out, v_out,
                                capacity_rows, lengths, offsets, arena, check=True) -> int:
    """Lists of host tensors, one entry per layer; ``arena`` is a device tensor."""
    c = p.c_struct()
    n = len(k)
    arrays = [_ptr_array(x) for x in (q_win, k, v, k_out, v_out, lengths, offsets)]
    rc = lib().refree_compress_layers_host(ctypes.byref(c), n, arrays[0], arrays[1], arrays[2], k[0].numel(),
                                           _dp(seq_start), _dp(seq_len), total_tokens, arrays[3], arrays[4],
                                           capacity_rows, arrays[5], arrays[6], _dp(arena),
                                           arena.numel() * arena.element_size())
    if check:
        _check(rc, "refree_compress_layers_host")
    return rc


def refree_sol_read_stream(src: torch.Tensor, stream=None, bulk=False) -> None:
    """Read every byte of ``src`` once (memory-system probe; ``bulk``: through the bulk-copy engine)."""
    _check(lib().refree_sol_read_stream(_dp(src), ctypes.c_int64(src.numel() * src.element_size()),
                                        ctypes.c_void_p(1) if bulk else None, _stream(stream)), "refree_sol_read_stream")


def refree_sol_row_mix(k, v, k_out, v_out, rows: int, kept_rows: int, row_bytes: int, stream=None, bulk=False) -> None:
    """Read ``rows`` rows of ``k``; copy the last ``kept_rows`` rows of ``k`` and ``v`` (memory-system probe)."""
    _check(lib().refree_sol_row_mix(_dp(k), _dp(v), _dp(k_out), _dp(v_out), ctypes.c_int64(rows), ctypes.c_int64(kept_rows),
                                    ctypes.c_int32(row_bytes), ctypes.c_void_p(1) if bulk else None, _stream(stream)),
           "refree_sol_row_mix")


def refree_layers_workspace_size(p: Params, total_tokens: int) -> int:
    out = _SZ(0)
    c = p.c_struct()
    _check(lib().refree_layers_workspace_size(ctypes.byref(c), total_tokens, ctypes.byref(out)),
           "refree_layers_workspace_size")
    return int(out.value)


class LayerPointers:
    """The seven per-layer pointer arrays of ``refree_compress_layers``, built once for lists of device
    tensors (one entry per layer) so that repeated calls marshal nothing."""

    def __init__(self, q_win, k, v, k_out, v_out, lengths, offsets):
        self.num_layers = len(k)
        self.keep = (q_win, k, v, k_out, v_out, lengths, offsets)
        self.arrays = [_ptr_array(x) for x in self.keep]


def refree_compress_layers(p: Params, ptrs: LayerPointers, seq_start, seq_len, total_tokens, capacity_rows,
                           workspace, device_status=None, stream=None, check=True) -> int:
    c = p.c_struct()
    a = ptrs.arrays
    rc = lib().refree_compress_layers(ctypes.byref(c), ptrs.num_layers, a[0], a[1], a[2], _dp(seq_start), _dp(seq_len),
                                      total_tokens, a[3], a[4], capacity_rows, a[5], a[6], _dp(workspace),
                                      workspace.numel() * workspace.element_size() if workspace is not None else 0,
                                      _dp(device_status), _stream(stream))
    if check:
        _check(rc, "refree_compress_layers")
    return rc


@dataclasses.dataclass
class LayerResult:
    k_out: torch.Tensor
    v_out: torch.Tensor
    lengths: torch.Tensor     # int32 [B, Hkv]
    offsets: torch.Tensor     # int64 [B*Hkv + 1]
    kept_idx: Optional[torch.Tensor]
    scores: Optional[torch.Tensor]
    device_status: torch.Tensor


def params_for(cfg, layer_cache, **overrides) -> Params:
    """``Params`` for a ``workloads.LayerCache`` (strides in elements)."""
    ss, st, sh = layer_cache.strides()
    p = Params(num_seqs=int(layer_cache.seq_len.numel()), num_q_heads=cfg.num_q_heads,
               num_kv_heads=cfg.num_kv_heads, head_dim=cfg.head_dim, window=cfg.window, sink=cfg.sink,
               dtype=DTYPE_F32 if cfg.dtype == "fp32" else DTYPE_BF16,
               kv_tokens=layer_cache.total_tokens, k_strides=(ss, st, sh), v_strides=(ss, st, sh))
    for key, val in overrides.items():
        setattr(p, key, val)
    return p


def compress_layer(p: Params, q_win, k, v, seq_start, seq_len, total_tokens, want_scores=True,
                   want_kept_idx=True, capacity_rows=None, workspace=None, stream=None) -> LayerResult:
    """Allocate outputs with torch and run the fused pass on device tensors."""
    dev = k.device
    cap = p.num_kv_heads * total_tokens if capacity_rows is None else capacity_rows
    k_out = torch.empty(max(cap, 1), p.head_dim, dtype=k.dtype, device=dev)
    v_out = torch.empty(max(cap, 1), p.head_dim, dtype=v.dtype, device=dev)
    units = p.num_seqs * p.num_kv_heads
    lengths = torch.zeros(units, dtype=torch.int32, device=dev)
    offsets = torch.zeros(units + 1, dtype=torch.int64, device=dev)
    kept = torch.empty(max(cap, 1), dtype=torch.int32, device=dev) if want_kept_idx else None
    scores = torch.empty(p.num_kv_heads, total_tokens, dtype=torch.float32, device=dev) if want_scores else None
    if workspace is None:
        workspace = torch.empty(refree_workspace_size(p, total_tokens), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    refree_compress_layer(p, q_win, k, v, seq_start, seq_len, total_tokens, k_out, v_out, cap, lengths, offsets,
                          kept, scores, workspace, status, stream)
    return LayerResult(k_out, v_out, lengths.view(p.num_seqs, p.num_kv_heads), offsets, kept, scores, status)
