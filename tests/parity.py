"""Helpers of the GPU parity tests: run the oracle and the CUDA library on the
same seeded layer and compare them under the acceptance rules.

Acceptance (written here once, used by every parity test):
  scores    |gpu - oracle| <= 1e-3 * |oracle| + 1e-9 * max(oracle)
  budgets   equal; a difference is tolerated only at a documented near-tie: every
            rank j between the two budgets has |sqrt(C_j/C_n) - (1 - T)| < 1e-6
            on the oracle's own criterion curve
  kept set  position ranking: a function of the budget (prefix + suffix), checked
            as such; score ranking: equal, except swaps between positions whose
            oracle scores differ by less than 1e-6 relative
  K_c, V_c  bit-identical to the source rows named by kept_idx; bit-identical to
            the oracle's output wherever the kept sets agree
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import refree_oracle as orc
from paper_2502_16886_b200 import binding

SCORE_RTOL = 1e-3
SCORE_ATOL_OF_MAX = 1e-9
TIE_TOL = 1e-6


def oracle_params(p: binding.Params) -> orc.OracleParams:
    return orc.OracleParams(p.num_seqs, p.num_q_heads, p.num_kv_heads, p.head_dim, window=p.window,
                            sink=p.sink, threshold=p.threshold, rank_mode=p.rank_mode, scope=p.scope,
                            keep_window=p.keep_window, force_full=p.force_full, dtype=p.dtype,
                            k_strides=p.k_strides, v_strides=p.v_strides)


def bits(t: torch.Tensor) -> torch.Tensor:
    return t.view(torch.int32) if t.dtype == torch.float32 else t.view(torch.int16)


def check_scores(gpu_scores: torch.Tensor, want: np.ndarray):
    got = gpu_scores.detach().cpu().double().numpy()
    assert np.isfinite(got).all()
    tol = SCORE_RTOL * np.abs(want) + SCORE_ATOL_OF_MAX * want.max(initial=0.0)
    err = np.abs(got - want)
    bad = err > tol
    assert not bad.any(), (f"{bad.sum()} scores out of tolerance; worst rel "
                           f"{(err / np.maximum(np.abs(want), 1e-300)).max():.3e}")
    return float((err / np.maximum(np.abs(want), 1e-300))[want > 1e-9 * want.max(initial=0.0)].max(initial=0.0))


def check_selection(p: binding.Params, seq_len, lengths, offsets, kept_idx, sel: orc.Selection,
                    scores_ref: np.ndarray, tie_tol: float = TIE_TOL):
    """Budgets, offsets and kept sets of the CUDA path against the oracle's selection.
    Returns the number of units accepted under the near-tie rule."""
    lengths = lengths.detach().cpu().numpy().reshape(p.num_seqs, p.num_kv_heads)
    offsets = offsets.detach().cpu().numpy()
    kept_idx = None if kept_idx is None else kept_idx.detach().cpu().numpy()
    seq_len = np.asarray(seq_len).reshape(-1)
    np.testing.assert_array_equal(offsets, np.concatenate([[0], np.cumsum(lengths.reshape(-1))]))
    T = float(np.float32(p.threshold))
    ties = 0
    pack = np.concatenate([[0], np.cumsum(seq_len)])
    for s in range(p.num_seqs):
        n = int(seq_len[s])
        w_eff, lead = min(p.window, n), min(p.sink, n)
        for g in range(p.num_kv_heads):
            u = s * p.num_kv_heads + g
            bg, bo = int(lengths[s, g]), int(sel.lengths[s, g])
            assert 0 <= bg <= n
            if bg != bo:
                lo, hi = min(bg, bo), max(bg, bo)
                curve = sel.ratio[g, pack[s] + max(lo, 1) - 1: pack[s] + hi]
                assert lo >= 1 and (np.abs(curve - (1.0 - T)) < tie_tol).all(), \
                    f"unit (s={s}, g={g}): budget {bg} vs oracle {bo} is not a near-tie"
                ties += 1
            if kept_idx is None:
                continue
            kept = kept_idx[offsets[u]: offsets[u + 1]]
            assert len(kept) == bg
            assert (np.diff(kept) > 0).all() and (bg == 0 or (kept[0] >= 0 and kept[-1] < n))
            if p.keep_window and not p.force_full:
                assert set(range(n - w_eff, n)) <= set(kept.tolist())
            if p.rank_mode == binding.RANK_POSITION or p.force_full:
                head = min(bg, lead)
                want = np.concatenate([np.arange(head), np.arange(n - (bg - head), n)])
                np.testing.assert_array_equal(kept, want)
            elif bg == bo:
                ref = sel.kept_idx[sel.offsets[u]: sel.offsets[u + 1]]
                if not np.array_equal(kept, ref):
                    only_g = np.setdiff1d(kept, ref)
                    only_o = np.setdiff1d(ref, kept)
                    assert len(only_g) == len(only_o)
                    if p.scope == binding.SCOPE_HEAD:
                        key = scores_ref[g, pack[s]: pack[s] + n].astype(np.float64) ** 2
                    else:
                        key = (scores_ref[:, pack[s]: pack[s] + n].astype(np.float64) ** 2).sum(axis=0)
                    a, b = np.sort(key[only_g]), np.sort(key[only_o])
                    assert (np.abs(a - b) <= 2 * tie_tol * np.maximum(a, b)).all(), \
                        f"unit (s={s}, g={g}): kept sets differ beyond score near-ties"
                    ties += 1
    return ties


def check_compaction(p: binding.Params, lay, lengths, offsets, kept_idx, k_out, v_out, ref=None):
    """Every output row is the bit copy of the source row kept_idx names."""
    lengths = lengths.detach().cpu().numpy().reshape(-1)
    offsets = offsets.detach().cpu().numpy()
    kept_idx = kept_idx.detach().cpu().numpy()
    k_out, v_out = k_out.detach().cpu(), v_out.detach().cpu()
    k_src, v_src = lay.k, lay.v
    if lay.layout == "token_major":
        k_src, v_src = k_src.permute(1, 0, 2), v_src.permute(1, 0, 2)
    for s in range(p.num_seqs):
        for g in range(p.num_kv_heads):
            u = s * p.num_kv_heads + g
            idx = torch.from_numpy(kept_idx[offsets[u]: offsets[u + 1]].astype(np.int64)) + int(lay.seq_start[s])
            assert torch.equal(bits(k_out[offsets[u]: offsets[u + 1]]), bits(k_src[g, idx]))
            assert torch.equal(bits(v_out[offsets[u]: offsets[u + 1]]), bits(v_src[g, idx]))
    if ref is not None and np.array_equal(lengths, ref.sel.lengths.reshape(-1)) and \
            np.array_equal(kept_idx[: offsets[-1]], ref.sel.kept_idx):
        assert torch.equal(bits(k_out[: offsets[-1]]), bits(ref.k_out))
        assert torch.equal(bits(v_out[: offsets[-1]]), bits(ref.v_out))


def run_fused_and_check(cfg, lay, want_scores=True, **overrides):
    """One layer through refree_compress_layer and through the oracle; all checks."""
    p = binding.params_for(cfg, lay, **overrides)
    dev = torch.device("cuda:0")
    total = lay.total_tokens
    res = binding.compress_layer(p, lay.q_win.to(dev), lay.k.to(dev), lay.v.to(dev), lay.seq_start.to(dev),
                                 lay.seq_len.to(dev), total, want_scores=want_scores)
    torch.cuda.synchronize()
    assert int(res.device_status.item()) == 0
    ref = orc.compress_layer(oracle_params(p), lay.q_win, lay.k, lay.v, lay.seq_start, lay.seq_len)
    worst = check_scores(res.scores, ref.scores) if want_scores and not p.force_full else 0.0
    ties = check_selection(p, lay.seq_len.numpy(), res.lengths, res.offsets, res.kept_idx, ref.sel, ref.scores32)
    check_compaction(p, lay, res.lengths, res.offsets, res.kept_idx, res.k_out, res.v_out, ref)
    return res, ref, worst, ties
