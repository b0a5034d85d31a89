"""Seeded synthetic prefill caches for the post-prefill KV-compression pass.

This module only draws random numbers and lays tensors out in memory.  It holds
none of the method's arithmetic (no softmax, no ranking, no stopping rule), so
the CPU oracle and the CUDA path can both be fed from it without sharing any
code of the method itself.

The paper evaluates on long-document and short-reasoning prompts run through
trained models (Section 4.1); neither the datasets nor the weights are used
here.  The stand-in is a Gaussian cache with a controlled set of "heavy"
positions and an attention sink, which reproduces the two properties the pass
is sensitive to: a small set of positions holding most of the attention mass,
and a first position that dominates it (the attention-sink observation the
paper builds its position ranking on, Section 3.2 "Initial Ranking").

Recipe for one (config c, layer l, sequence s), all draws from a CPU
``torch.Generator`` seeded ``1_000_000*c + 1000*l + s`` (config 0 uses seed 0),
in this order, in fp32, then rounded once to the storage dtype:

1. ``K[g, i, :]`` ~ N(0, 1), shape ``[Hkv, n, d]``.
2. ``V[g, i, :]`` ~ N(0, 1), same shape.
3. ``mu[g, :]`` ~ N(0, I_d), one window direction per KV head;
   ``u[g] = mu[g] / |mu[g]|``.
4. ``z[h, r, :]`` ~ N(0, 1), shape ``[Hq, w, d]``; the window queries are
   ``q[h, r] = (z[h, r] + mu[g(h)]) / sqrt(2)`` (unit-variance coordinates with
   a mean shared by the query group, so that "aligned with the window queries"
   means something for every row of the window).
5. heavy positions: per KV head, ``n_heavy`` indices without replacement from
   ``[sink, n - w)`` (``torch.randperm`` of that range, first ``n_heavy``);
   ``K[g, i] += heavy_scale * sqrt(2) * u[g]`` which lifts the logit of those
   positions by about ``heavy_scale``.
6. attention sink: ``K[g, 0] += sink_scale * sqrt(2) * u[g]`` when the config
   has one.

Sequence lengths and per-sequence heavy fractions of the ragged config come
from a generator seeded ``1_000_000*c + 999_999`` (the same for every layer).
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import torch


@dataclasses.dataclass(frozen=True)
class CacheConfig:
    """Shape of one synthetic prefill cache (one entry per benchmark config)."""

    name: str
    index: int                 # position in the config list; part of the seed
    num_layers: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    window: int
    dtype: str                 # "fp32" | "bf16"
    seq_lens: Optional[tuple]  # fixed lengths, or None when drawn per config
    num_seqs: int = 1
    len_range: Optional[tuple] = None      # inclusive range for drawn lengths
    heavy_count: Optional[int] = None      # fixed number of heavy positions
    heavy_fracs: tuple = ()                # cycled by layer when non-empty
    heavy_frac_range: Optional[tuple] = None  # drawn per sequence
    heavy_scale: float = 3.0
    sink_scale: float = 0.0
    sink: int = 4              # protected leading positions m of the ranking

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "fp32" else 2


CONFIGS: List[CacheConfig] = [
    CacheConfig("tiny", 0, 1, 4, 2, 64, 32, "fp32", (512,),
                heavy_count=8, heavy_scale=4.0, sink_scale=0.0),
    CacheConfig("llama3_8b_8k", 1, 32, 32, 8, 128, 64, "bf16", (8192,),
                heavy_fracs=(0.01,), heavy_scale=3.0, sink_scale=6.0),
    CacheConfig("mistral7b_32k", 2, 32, 32, 8, 128, 64, "bf16", (32768,),
                heavy_fracs=(0.005, 0.02, 0.05), heavy_scale=3.0, sink_scale=6.0),
    CacheConfig("qwen25_7b_ragged8", 3, 28, 28, 4, 128, 64, "bf16", None,
                num_seqs=8, len_range=(2048, 16384),
                heavy_frac_range=(0.005, 0.05), heavy_scale=3.0, sink_scale=6.0),
    CacheConfig("llama3_70b_20k", 4, 80, 64, 8, 128, 64, "bf16", (20480,),
                heavy_fracs=(0.01,), heavy_scale=3.0, sink_scale=6.0),
]


def get_config(name: str) -> CacheConfig:
    for c in CONFIGS:
        if c.name == name:
            return c
    raise KeyError(f"unknown workload {name!r}; have {[c.name for c in CONFIGS]}")


def _config_draws(cfg: CacheConfig):
    """Per-config draws shared by every layer: sequence lengths, heavy fractions."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(1_000_000 * cfg.index + 999_999)
    if cfg.seq_lens is not None:
        lens = list(cfg.seq_lens)
    else:
        lo, hi = cfg.len_range
        lens = torch.randint(lo, hi + 1, (cfg.num_seqs,), generator=gen).tolist()
    if cfg.heavy_frac_range is not None:
        lo, hi = cfg.heavy_frac_range
        fr = (lo + (hi - lo) * torch.rand(len(lens), generator=gen, dtype=torch.float64)).tolist()
    else:
        fr = [None] * len(lens)
    return lens, fr


def sequence_lengths(cfg: CacheConfig) -> List[int]:
    return _config_draws(cfg)[0]


def heavy_count(cfg: CacheConfig, layer: int, seq: int, n: int) -> int:
    """Number of heavy positions per KV head for this (layer, sequence)."""
    if cfg.heavy_count is not None:
        cnt = cfg.heavy_count
    elif cfg.heavy_frac_range is not None:
        cnt = math.ceil(_config_draws(cfg)[1][seq] * n)
    else:
        cnt = math.ceil(cfg.heavy_fracs[layer % len(cfg.heavy_fracs)] * n)
    return max(0, min(cnt, n - cfg.window - cfg.sink))


@dataclasses.dataclass
class LayerCache:
    """One layer of a synthetic cache, CPU tensors in the storage dtype.

    ``k``/``v`` are ``[Hkv, N, d]`` (head-major, sequences packed back to back
    along the token axis) or ``[N, Hkv, d]`` when ``layout == "token_major"``.
    Element ``(s, g, i, :)`` lives at
    ``s*stride_seq + (seq_start[s] + i)*stride_tok + g*stride_head`` (elements).
    """

    cfg: CacheConfig
    layer: int
    layout: str
    q_win: torch.Tensor        # [B, Hq, w, d]
    k: torch.Tensor
    v: torch.Tensor
    seq_start: torch.Tensor    # int32 [B]
    seq_len: torch.Tensor      # int32 [B]
    heavy_idx: list            # per sequence: LongTensor [Hkv, n_heavy]

    @property
    def total_tokens(self) -> int:
        return int(self.seq_len.sum().item())

    def strides(self):
        """(stride_seq, stride_tok, stride_head) in elements, same for K and V."""
        d, hkv, n = self.cfg.head_dim, self.cfg.num_kv_heads, self.total_tokens
        if self.layout == "head_major":
            return 0, d, n * d
        return 0, hkv * d, d


def make_layer(cfg: CacheConfig, layer: int, layout: str = "head_major",
               seq_lens: Optional[List[int]] = None) -> LayerCache:
    """Draw layer ``layer`` of config ``cfg``.  ``seq_lens`` overrides the
    config's lengths (used by tests for ragged tails and degenerate sizes)."""
    if layout not in ("head_major", "token_major"):
        raise ValueError(layout)
    lens = list(seq_lens) if seq_lens is not None else sequence_lengths(cfg)
    hq, hkv, d, w = cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, cfg.window
    grp = cfg.group
    total = sum(lens)
    k_all = torch.empty(hkv, total, d, dtype=cfg.torch_dtype)
    v_all = torch.empty(hkv, total, d, dtype=cfg.torch_dtype)
    q_all = torch.empty(len(lens), hq, w, d, dtype=cfg.torch_dtype)
    heavy_all = []
    start = 0
    starts = []
    for s, n in enumerate(lens):
        gen = torch.Generator(device="cpu")
        gen.manual_seed(0 if cfg.index == 0 else 1_000_000 * cfg.index + 1000 * layer + s)
        k = torch.randn(hkv, n, d, generator=gen, dtype=torch.float32)
        v = torch.randn(hkv, n, d, generator=gen, dtype=torch.float32)
        mu = torch.randn(hkv, d, generator=gen, dtype=torch.float32)
        z = torch.randn(hq, w, d, generator=gen, dtype=torch.float32)
        u = mu / mu.norm(dim=-1, keepdim=True)
        q = (z + mu.repeat_interleave(grp, dim=0)[:, None, :]) / math.sqrt(2.0)
        cnt = heavy_count(cfg, layer, s, n) if seq_lens is None else \
            max(0, min(cfg.heavy_count or math.ceil(0.01 * n), n - w - cfg.sink))
        idx = torch.empty(hkv, cnt, dtype=torch.long)
        span = n - w - cfg.sink
        for g in range(hkv):
            if cnt > 0:
                idx[g] = cfg.sink + torch.randperm(span, generator=gen)[:cnt]
                k[g, idx[g]] += cfg.heavy_scale * math.sqrt(2.0) * u[g]
            if cfg.sink_scale > 0 and n > 0:
                k[g, 0] += cfg.sink_scale * math.sqrt(2.0) * u[g]
        k_all[:, start:start + n] = k.to(cfg.torch_dtype)
        v_all[:, start:start + n] = v.to(cfg.torch_dtype)
        q_all[s] = q.to(cfg.torch_dtype)
        heavy_all.append(idx)
        starts.append(start)
        start += n
    if layout == "token_major":
        k_all = k_all.permute(1, 0, 2).contiguous()
        v_all = v_all.permute(1, 0, 2).contiguous()
    return LayerCache(cfg, layer, layout, q_all, k_all, v_all,
                      torch.tensor(starts, dtype=torch.int32),
                      torch.tensor(lens, dtype=torch.int32), heavy_all)


def make_decode_query(cfg: CacheConfig, layer: int, q_win: torch.Tensor) -> torch.Tensor:
    """Query of the first generated token, ``[B, Hq, d]`` in the cache dtype.

    Drawn like a window row (unit-variance coordinates around the direction the
    window queries of the head share, estimated here as their mean over the
    window), from a generator seeded ``1_000_000*c + 1000*layer + 777``.
    """
    gen = torch.Generator(device="cpu")
    gen.manual_seed(1_000_000 * cfg.index + 1000 * layer + 777)
    mean = q_win.to(torch.float32).mean(dim=2)                      # [B, Hq, d]
    z = torch.randn(mean.shape, generator=gen, dtype=torch.float32)
    return (z / math.sqrt(2.0) + mean).to(cfg.torch_dtype).contiguous()


def make_ragged_cache(seed: int, lengths, head_dim: int, dtype: torch.dtype):
    """A dense ragged cache with the given per-unit row counts (rows ~ N(0,1)):
    ``(k_c, v_c, offsets)`` with ``offsets`` the int64 running sum of ``lengths``."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    rows = int(sum(lengths))
    k_c = torch.randn((max(rows, 1), head_dim), generator=gen, dtype=torch.float32).to(dtype)
    v_c = torch.randn((max(rows, 1), head_dim), generator=gen, dtype=torch.float32).to(dtype)
    offsets = torch.zeros(len(lengths) + 1, dtype=torch.int64)
    offsets[1:] = torch.cumsum(torch.tensor(list(lengths), dtype=torch.int64), 0)
    return k_c, v_c, offsets
