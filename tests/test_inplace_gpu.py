"""In-place compaction (refree_compact_inplace) against the oracle.

The oracle's selection (budgets, offsets, kept positions) and its dense compacted
cache are computed on the CPU; the kernel is then given the oracle's selection and
must leave, at the front (or, for position ranking, optionally at the end) of every
unit's own region of K and V, exactly the rows the oracle compacted (bit compare).
Sizes span several rounds of the front-anchored kernel (one round is what the whole
grid holds in registers, about 38 K rows of 256 bytes) and ragged tails; both
rankings, both layouts, both storage types.
"""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import refree_oracle as orc
from paper_2502_16886_b200 import binding, build, workloads
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    binding.lib()


def _cfg(**kw):
    return dataclasses.replace(workloads.CONFIGS[0], **kw)


def _unit_rows(t, lay, s, g, count, back=False):
    """First (or, ``back``, last) ``count`` rows of unit (s, g)'s own region of a cache tensor laid out like ``lay``."""
    view = t.permute(1, 0, 2) if lay.layout == "token_major" else t
    a = int(lay.seq_start[s])
    if back:
        a += int(lay.seq_len[s]) - count
    return view[g, a:a + count]


def _selection(p, lay, rng, power):
    """Oracle selection from synthetic fp32 scores (the stage under test moves rows, it does not score)."""
    total = lay.total_tokens
    scores = (rng.random((p.num_kv_heads, total)) ** power).astype(np.float32)
    return orc.select(parity.oracle_params(p), scores, lay.seq_len)


def _run_inplace_and_check(p, lay, sel, anchor=binding.ANCHOR_FRONT):
    op = parity.oracle_params(p)
    want_k, want_v = orc.compact(op, lay.k, lay.v, lay.seq_start, lay.seq_len, sel)
    k, v = lay.k.to(DEV), lay.v.to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    offsets = torch.from_numpy(sel.offsets).to(DEV)
    kept = torch.from_numpy(sel.kept_idx if sel.kept_idx.size else np.zeros(1, np.int32)).to(DEV)
    ranges = p.rank_mode == binding.RANK_POSITION or p.force_full
    binding.refree_compact_inplace(p, k, v, lay.seq_start.to(DEV), lay.seq_len.to(DEV), offsets,
                                   None if ranges else kept, status, anchor=anchor)
    torch.cuda.synchronize()
    assert status.item() == 0
    k, v = k.cpu(), v.cpu()
    moved = 0
    back = anchor == binding.ANCHOR_BACK
    for s in range(p.num_seqs):
        for g in range(p.num_kv_heads):
            u = s * p.num_kv_heads + g
            a, b = int(sel.offsets[u]), int(sel.offsets[u + 1])
            assert b - a == int(sel.lengths[s, g])
            assert torch.equal(parity.bits(_unit_rows(k, lay, s, g, b - a, back)), parity.bits(want_k[a:b]))
            assert torch.equal(parity.bits(_unit_rows(v, lay, s, g, b - a, back)), parity.bits(want_v[a:b]))
            moved += b - a
    return moved


@pytest.mark.parametrize("rank_mode", [binding.RANK_POSITION, binding.RANK_SCORE])
@pytest.mark.parametrize("layout,dtype,d", [("head_major", "bf16", 128), ("token_major", "bf16", 128),
                                            ("head_major", "fp32", 64), ("token_major", "fp32", 128)])
def test_inplace_compaction_matches_the_oracle_over_several_rounds(rank_mode, layout, dtype, d):
    cfg = _cfg(window=16, dtype=dtype, head_dim=d, num_q_heads=4, num_kv_heads=2)
    lay = workloads.make_layer(cfg, 1, layout=layout, seq_lens=[61000, 90, 0, 14001, 1])
    p = binding.params_for(cfg, lay, rank_mode=rank_mode, threshold=0.02)
    sel = _selection(p, lay, np.random.default_rng(5), power=3)
    moved = _run_inplace_and_check(p, lay, sel)
    assert 45000 < moved < 2 * lay.total_tokens       # more than one round, and something was dropped


@pytest.mark.parametrize("rank_mode", [binding.RANK_POSITION, binding.RANK_SCORE])
def test_inplace_compaction_small_budgets_and_short_sequences(rank_mode):
    # a high threshold keeps little (long moves, no overlap of source and destination); lengths around the
    # sink and window sizes exercise the floor
    cfg = _cfg(window=8, dtype="bf16", head_dim=128, num_q_heads=6, num_kv_heads=3)
    lay = workloads.make_layer(cfg, 0, seq_lens=[3, 4, 5, 12, 13, 700, 2049])
    p = binding.params_for(cfg, lay, rank_mode=rank_mode, threshold=0.6)
    _run_inplace_and_check(p, lay, _selection(p, lay, np.random.default_rng(6), power=8))


@pytest.mark.parametrize("layout,dtype,d", [("head_major", "bf16", 128), ("token_major", "bf16", 128),
                                            ("head_major", "fp32", 64)])
@pytest.mark.parametrize("sink,threshold", [(4, 0.02), (4, 0.6), (0, 0.1), (40, 0.3), (700, 0.05)])
def test_inplace_anchored_at_the_end_lifts_only_the_leading_rows(layout, dtype, d, sink, threshold):
    """Position ranking, compacted cache in rows [n - b, n): against the oracle's dense output.  Sink counts
    from none to more rows than one block of the kernel moves at once, budgets that make the lifted rows
    overlap their own sources (n - b < sink) and budgets that do not."""
    cfg = _cfg(window=8, dtype=dtype, head_dim=d, num_q_heads=4, num_kv_heads=2, sink=sink)
    lay = workloads.make_layer(cfg, 2, layout=layout, seq_lens=[5000, 3, 0, 41, 709, 1, 2300])
    p = binding.params_for(cfg, lay, threshold=threshold)
    sel = _selection(p, lay, np.random.default_rng(11), power=4)
    shifts = [int(n) - int(b) for n, row in zip(lay.seq_len.tolist(), sel.lengths.tolist()) for b in row]
    assert any(x > 0 for x in shifts)
    if sink == 700:
        assert any(0 < x < 700 for x in shifts)      # a self-overlapping move of several blocks
    _run_inplace_and_check(p, lay, sel, anchor=binding.ANCHOR_BACK)


def test_inplace_anchored_at_the_end_is_for_position_ranking_only():
    cfg = _cfg(window=8, dtype="bf16", head_dim=128, num_q_heads=2, num_kv_heads=1)
    lay = workloads.make_layer(cfg, 0, seq_lens=[100])
    p = binding.params_for(cfg, lay, rank_mode=binding.RANK_SCORE)
    k, v = lay.k.to(DEV), lay.v.to(DEV)
    off = torch.tensor([0, 50], dtype=torch.int64, device=DEV)
    kept = torch.arange(50, dtype=torch.int32, device=DEV)
    rc = binding.refree_compact_inplace(p, k, v, lay.seq_start.to(DEV), lay.seq_len.to(DEV), off, kept, check=False,
                                        anchor=binding.ANCHOR_BACK)
    assert rc == binding.ERR_UNSUPPORTED
    assert binding.refree_compact_inplace(p, k, v, lay.seq_start.to(DEV), lay.seq_len.to(DEV), off, kept, check=False,
                                          anchor=7) == binding.ERR_INVALID_ARG


def test_inplace_compaction_of_a_frozen_layer_changes_nothing():
    cfg = _cfg(window=8, dtype="bf16", head_dim=128, num_q_heads=4, num_kv_heads=2)
    lay = workloads.make_layer(cfg, 0, seq_lens=[900, 31])
    p = binding.params_for(cfg, lay, force_full=1)
    sel = _selection(p, lay, np.random.default_rng(7), power=2)
    assert sel.lengths.reshape(-1).tolist() == [900, 900, 31, 31]
    k, v = lay.k.to(DEV), lay.v.to(DEV)
    binding.refree_compact_inplace(p, k, v, lay.seq_start.to(DEV), lay.seq_len.to(DEV),
                                   torch.from_numpy(sel.offsets).to(DEV), None)
    torch.cuda.synchronize()
    assert torch.equal(parity.bits(k.cpu()), parity.bits(lay.k)) and torch.equal(parity.bits(v.cpu()), parity.bits(lay.v))


def test_inplace_after_the_library_selection_equals_the_out_of_place_pass():
    """Whole pass on the GPU: score and select through the C ABI, then once out of place and once in place."""
    cfg = _cfg(window=16, dtype="bf16", head_dim=128, num_q_heads=8, num_kv_heads=2)
    lay = workloads.make_layer(cfg, 3, seq_lens=[5000, 257])
    for rank_mode in (binding.RANK_POSITION, binding.RANK_SCORE):
        p = binding.params_for(cfg, lay, rank_mode=rank_mode, threshold=0.05)
        q, k, v, ss, sl = [t.to(DEV) for t in (lay.q_win, lay.k, lay.v, lay.seq_start, lay.seq_len)]
        res = binding.compress_layer(p, q, k, v, ss, sl, lay.total_tokens)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        binding.refree_compact_inplace(p, k, v, ss, sl, res.offsets, res.kept_idx, status)
        torch.cuda.synchronize()
        assert status.item() == 0 and res.device_status.item() == 0
        off = res.offsets.cpu().tolist()
        kc, vc = k.cpu(), v.cpu()
        for s in range(p.num_seqs):
            for g in range(p.num_kv_heads):
                u = s * p.num_kv_heads + g
                assert 0 < off[u + 1] - off[u] <= int(lay.seq_len[s])
                assert torch.equal(parity.bits(_unit_rows(kc, lay, s, g, off[u + 1] - off[u])),
                                   parity.bits(res.k_out[off[u]:off[u + 1]].cpu()))
                assert torch.equal(parity.bits(_unit_rows(vc, lay, s, g, off[u + 1] - off[u])),
                                   parity.bits(res.v_out[off[u]:off[u + 1]].cpu()))


@pytest.mark.parametrize("rank_mode,anchor,window,dtype", [
    (binding.RANK_POSITION, binding.ANCHOR_BACK, 16, "bf16"), (binding.RANK_POSITION, binding.ANCHOR_FRONT, 16, "bf16"),
    (binding.RANK_SCORE, binding.ANCHOR_FRONT, 16, "bf16"), (binding.RANK_POSITION, binding.ANCHOR_BACK, 1, "bf16"),
    (binding.RANK_POSITION, binding.ANCHOR_BACK, 8, "fp32")])
def test_fused_inplace_pass_against_the_oracle(rank_mode, anchor, window, dtype):
    """refree_compress_layer_inplace: budgets equal to the oracle's and, in every unit's own region, the rows
    of the oracle's dense compacted cache (tensor-core, single-row and generic scoring paths)."""
    cfg = _cfg(window=window, dtype=dtype, head_dim=128, num_q_heads=8, num_kv_heads=2)
    lay = workloads.make_layer(cfg, 4, seq_lens=[3000, 130, 0, 777])
    p = binding.params_for(cfg, lay, rank_mode=rank_mode, threshold=0.05)
    ref = orc.compress_layer(parity.oracle_params(p), lay.q_win, lay.k, lay.v, lay.seq_start, lay.seq_len)
    q, k, v, ss, sl = [t.to(DEV) for t in (lay.q_win, lay.k, lay.v, lay.seq_start, lay.seq_len)]
    units = p.num_seqs * p.num_kv_heads
    lengths = torch.zeros(units, dtype=torch.int32, device=DEV)
    offsets = torch.zeros(units + 1, dtype=torch.int64, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = torch.empty(binding.refree_workspace_size(p, lay.total_tokens), dtype=torch.uint8, device=DEV)
    binding.refree_compress_layer_inplace(p, q, k, v, ss, sl, lay.total_tokens, lengths, offsets, anchor, ws, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert lengths.cpu().tolist() == ref.sel.lengths.reshape(-1).tolist()
    assert offsets.cpu().tolist() == ref.sel.offsets.tolist()
    kc, vc = k.cpu(), v.cpu()
    back = anchor == binding.ANCHOR_BACK
    for s in range(p.num_seqs):
        for g in range(p.num_kv_heads):
            u = s * p.num_kv_heads + g
            a, b = int(ref.sel.offsets[u]), int(ref.sel.offsets[u + 1])
            assert torch.equal(parity.bits(_unit_rows(kc, lay, s, g, b - a, back)), parity.bits(ref.k_out[a:b]))
            assert torch.equal(parity.bits(_unit_rows(vc, lay, s, g, b - a, back)), parity.bits(ref.v_out[a:b]))


@pytest.mark.parametrize("anchor", [binding.ANCHOR_BACK, binding.ANCHOR_FRONT])
@pytest.mark.parametrize("dtype,d,window", [("bf16", 128, 16), ("bf16", 64, 1), ("fp32", 128, 8)])
def test_decode_step_over_the_cache_compacted_in_place(anchor, dtype, d, window):
    """The in-place pass followed by one decode step that reads the strided ragged cache where it lies,
    against the oracle's dense compaction followed by the oracle's decode attention."""
    cfg = _cfg(window=window, dtype=dtype, head_dim=d, num_q_heads=8, num_kv_heads=2)
    lay = workloads.make_layer(cfg, 5, seq_lens=[2500, 130, 0, 4097, 1])
    p = binding.params_for(cfg, lay, threshold=0.05)
    op = parity.oracle_params(p)
    ref = orc.compress_layer(op, lay.q_win, lay.k, lay.v, lay.seq_start, lay.seq_len)
    q_new = workloads.make_decode_query(cfg, 5, lay.q_win)
    want = orc.decode_attention(op, q_new, ref.k_out, ref.v_out, ref.sel.offsets)
    q, k, v, ss, sl = [t.to(DEV) for t in (lay.q_win, lay.k, lay.v, lay.seq_start, lay.seq_len)]
    units = p.num_seqs * p.num_kv_heads
    lengths = torch.zeros(units, dtype=torch.int32, device=DEV)
    offsets = torch.zeros(units + 1, dtype=torch.int64, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = torch.empty(binding.refree_workspace_size(p, lay.total_tokens), dtype=torch.uint8, device=DEV)
    binding.refree_compress_layer_inplace(p, q, k, v, ss, sl, lay.total_tokens, lengths, offsets, anchor, ws, status)
    max_rows = int(lay.seq_len.max())
    dws = torch.empty(binding.refree_decode_workspace_size(p, max_rows), dtype=torch.uint8, device=DEV)
    out = torch.full((p.num_seqs, p.num_q_heads, d), float("nan"), dtype=torch.float32, device=DEV)
    binding.refree_decode_attention_inplace(p, q_new.to(DEV), k, v, ss, sl, lengths, anchor, max_rows, out, dws, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert lengths.cpu().tolist() == ref.sel.lengths.reshape(-1).tolist()
    got = out.cpu().numpy()
    assert np.isfinite(got).all()
    err = np.abs(got - want)
    assert (err <= 1e-4 + 1e-4 * np.abs(want)).all(), float(err.max())
    assert not got[2].any()                      # the empty sequence gives zero rows


def test_decode_over_the_in_place_cache_needs_head_major_rows():
    cfg = _cfg(window=8, dtype="bf16", head_dim=128, num_q_heads=4, num_kv_heads=2)
    lay = workloads.make_layer(cfg, 0, layout="token_major", seq_lens=[100])
    p = binding.params_for(cfg, lay)
    k, v, ss, sl = [t.to(DEV) for t in (lay.k, lay.v, lay.seq_start, lay.seq_len)]
    q_new = workloads.make_decode_query(cfg, 0, lay.q_win).to(DEV)
    lengths = torch.full((2,), 50, dtype=torch.int32, device=DEV)
    dws = torch.empty(binding.refree_decode_workspace_size(p, 100), dtype=torch.uint8, device=DEV)
    out = torch.zeros(1, 4, 128, dtype=torch.float32, device=DEV)
    rc = binding.refree_decode_attention_inplace(p, q_new, k, v, ss, sl, lengths, binding.ANCHOR_BACK, 100, out, dws,
                                                 check=False)
    assert rc == binding.ERR_UNSUPPORTED


def test_inplace_flags_offsets_that_do_not_fit_the_sequences():
    cfg = _cfg(window=8, dtype="bf16", head_dim=128, num_q_heads=2, num_kv_heads=1)
    lay = workloads.make_layer(cfg, 0, seq_lens=[100])
    p = binding.params_for(cfg, lay)
    k, v = lay.k.to(DEV), lay.v.to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    bad = torch.tensor([0, 101], dtype=torch.int64, device=DEV)        # budget above the sequence length
    binding.refree_compact_inplace(p, k, v, lay.seq_start.to(DEV), lay.seq_len.to(DEV), bad, None, status)
    torch.cuda.synchronize()
    assert status.item() & binding.DEV_CAPACITY
    assert torch.equal(parity.bits(k.cpu()), parity.bits(lay.k))      # nothing was moved
    # score ranking without an index list is refused on the host
    ps = binding.params_for(cfg, lay, rank_mode=binding.RANK_SCORE)
    assert binding.refree_compact_inplace(ps, k, v, lay.seq_start.to(DEV), lay.seq_len.to(DEV), bad, None,
                                          check=False) == binding.ERR_INVALID_ARG
