"""ctypes front end of the C oracle (``refree_oracle.c``).  Test infrastructure.

Takes CPU torch tensors (fp32 or bf16 storage) and numpy arrays, returns numpy
arrays.  Holds no arithmetic of its own beyond rounding the fp64 scores to fp32
at the stage boundary between scoring and selection, which is where the
compression pass defines its scores as fp32 values.
"""
from __future__ import annotations

import ctypes
import dataclasses

import numpy as np
import torch

from . import build as _build

_LIB = None


class _Params(ctypes.Structure):
    _fields_ = [
        ("num_seqs", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("window", ctypes.c_int32), ("sink", ctypes.c_int32),
        ("threshold", ctypes.c_double),
        ("rank_mode", ctypes.c_int32), ("scope", ctypes.c_int32),
        ("keep_window", ctypes.c_int32), ("force_full", ctypes.c_int32),
        ("dtype", ctypes.c_int32),
        ("k_stride_seq", ctypes.c_int64), ("k_stride_tok", ctypes.c_int64),
        ("k_stride_head", ctypes.c_int64),
        ("v_stride_seq", ctypes.c_int64), ("v_stride_tok", ctypes.c_int64),
        ("v_stride_head", ctypes.c_int64),
    ]


@dataclasses.dataclass
class OracleParams:
    num_seqs: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    window: int = 1            # paper default k = 1 (Section 4.1)
    sink: int = 4              # paper default m = 4 (Section 4.1)
    threshold: float = 0.01    # universal threshold T = 1 % (Section 3.2)
    rank_mode: int = 0         # 0 position ranking (paper default), 1 by score
    scope: int = 0             # 0 per (sequence, KV head), 1 per sequence
    keep_window: int = 1
    force_full: int = 0
    dtype: int = 1             # 0 fp32, 1 bf16
    k_strides: tuple = (0, 0, 0)   # (seq, tok, head) in elements
    v_strides: tuple = (0, 0, 0)

    def c_struct(self) -> _Params:
        # the threshold crosses the library boundary of the CUDA path as a C
        # float; the same fp32 value, widened, is the T used here
        t = float(np.float32(self.threshold))
        return _Params(self.num_seqs, self.num_q_heads, self.num_kv_heads, self.head_dim,
                       self.window, self.sink, t, self.rank_mode, self.scope,
                       self.keep_window, self.force_full, self.dtype,
                       *self.k_strides, *self.v_strides)


def lib():
    global _LIB
    if _LIB is None:
        _LIB = ctypes.CDLL(_build.build())
        _LIB.oracle_num_threads.restype = ctypes.c_int
    return _LIB


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_num_threads(t: int) -> None:
    lib().oracle_set_num_threads(ctypes.c_int(t))


def _raw(t: torch.Tensor) -> np.ndarray:
    """View a CPU tensor's storage bits as numpy (bf16 -> uint16)."""
    t = t.contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _i32(x) -> np.ndarray:
    if isinstance(x, torch.Tensor):
        x = x.numpy()
    return np.ascontiguousarray(x, dtype=np.int32)


def score(p: OracleParams, q_win, k, seq_start, seq_len) -> np.ndarray:
    """fp64 reduced attention ``[Hkv, total_tokens]`` (Eq. 2)."""
    seq_start, seq_len = _i32(seq_start), _i32(seq_len)
    total = int(seq_len.sum())
    out = np.zeros((p.num_kv_heads, total), dtype=np.float64)
    qa, ka = _raw(q_win), _raw(k)
    cs = p.c_struct()
    rc = lib().oracle_score(ctypes.byref(cs), _ptr(qa), _ptr(ka), _ptr(seq_start), _ptr(seq_len),
                            ctypes.c_int64(total), _ptr(out))
    assert rc == 0
    return out


@dataclasses.dataclass
class Selection:
    lengths: np.ndarray     # int32 [B, Hkv]
    offsets: np.ndarray     # int64 [B*Hkv + 1]
    kept_idx: np.ndarray    # int32 [sum lengths]
    pi: np.ndarray          # int32 [Hkv, total] ranked order per unit
    ratio: np.ndarray       # fp64 [Hkv, total] sqrt(C_j / C_n), j = 1..n
    gap: np.ndarray         # fp64 [B, Hkv] distance of the stop decision from a tie
    jstar: np.ndarray       # int32 [B, Hkv] stop index before the window floor


def select(p: OracleParams, scores32: np.ndarray, seq_len) -> Selection:
    """Stopping rule (Eq. 1 / Eq. 3) on fp32 scores ``[Hkv, total_tokens]``."""
    seq_len = _i32(seq_len)
    total = int(seq_len.sum())
    sc = np.ascontiguousarray(scores32, dtype=np.float32)
    assert sc.shape == (p.num_kv_heads, total)
    units = p.num_seqs * p.num_kv_heads
    lengths = np.zeros(units, dtype=np.int32)
    offsets = np.zeros(units + 1, dtype=np.int64)
    kept = np.zeros(max(1, units * max(1, int(seq_len.max(initial=0)))), dtype=np.int32)
    pi = np.zeros((p.num_kv_heads, total), dtype=np.int32)
    ratio = np.zeros((p.num_kv_heads, total), dtype=np.float64)
    gap = np.zeros(units, dtype=np.float64)
    jstar = np.zeros(units, dtype=np.int32)
    cs = p.c_struct()
    rc = lib().oracle_select(ctypes.byref(cs), _ptr(sc), _ptr(seq_len), ctypes.c_int64(total),
                             _ptr(lengths), _ptr(offsets), _ptr(kept), _ptr(pi), _ptr(ratio),
                             _ptr(gap), _ptr(jstar))
    assert rc == 0
    shape = (p.num_seqs, p.num_kv_heads)
    return Selection(lengths.reshape(shape), offsets, kept[: int(offsets[-1])].copy(), pi, ratio,
                     gap.reshape(shape), jstar.reshape(shape))


def compact(p: OracleParams, k, v, seq_start, seq_len, sel: Selection):
    """Dense ragged ``K_c, V_c`` (torch tensors ``[sum b, d]`` in the storage dtype)."""
    seq_start, seq_len = _i32(seq_start), _i32(seq_len)
    rows = int(sel.offsets[-1])
    k_out = torch.zeros(rows, p.head_dim, dtype=k.dtype)
    v_out = torch.zeros(rows, p.head_dim, dtype=v.dtype)
    ka, va, koa, voa = _raw(k), _raw(v), _raw(k_out), _raw(v_out)
    lengths = np.ascontiguousarray(sel.lengths.reshape(-1), dtype=np.int32)
    cs = p.c_struct()
    rc = lib().oracle_compact(ctypes.byref(cs), _ptr(ka), _ptr(va), _ptr(seq_start), _ptr(seq_len),
                              _ptr(lengths), _ptr(sel.offsets), _ptr(sel.kept_idx),
                              _ptr(koa), _ptr(voa))
    assert rc == 0
    return k_out, v_out


@dataclasses.dataclass
class Compressed:
    scores: np.ndarray      # fp64 [Hkv, total]
    scores32: np.ndarray    # the same rounded to fp32 (what selection consumes)
    sel: Selection
    k_out: torch.Tensor
    v_out: torch.Tensor


def compress_layer(p: OracleParams, q_win, k, v, seq_start, seq_len) -> Compressed:
    """The whole pass of Algorithm 1 for one layer: score, select, compact."""
    sc = score(p, q_win, k, seq_start, seq_len)
    sc32 = sc.astype(np.float32)
    sel = select(p, sc32, seq_len)
    k_out, v_out = compact(p, k, v, seq_start, seq_len, sel)
    return Compressed(sc, sc32, sel, k_out, v_out)


def decode_attention(p: OracleParams, q_new, k_c, v_c, offsets) -> np.ndarray:
    """One decode step over the compacted cache: fp64 ``[B, Hq, d]``."""
    out = np.zeros((p.num_seqs, p.num_q_heads, p.head_dim), dtype=np.float64)
    qa, ka, va = _raw(q_new), _raw(k_c), _raw(v_c)
    off = np.ascontiguousarray(offsets, dtype=np.int64)
    cs = p.c_struct()
    rc = lib().oracle_decode_attention(ctypes.byref(cs), _ptr(qa), _ptr(ka), _ptr(va), _ptr(off), _ptr(out))
    assert rc == 0
    return out
