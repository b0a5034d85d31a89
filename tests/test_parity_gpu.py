"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle
on the same seeded inputs (acceptance rules in ``tests/parity.py``)."""
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
def _built():
    build.build()
    binding.lib()


def small_cfg(**kw):
    """A reduced shape of the tiny config for sweeps (fp32, head_dim 64)."""
    return dataclasses.replace(workloads.CONFIGS[0], **kw)


# ------------------------------------------------------------ fused pass ----
@pytest.mark.parametrize("rank_mode", [binding.RANK_POSITION, binding.RANK_SCORE])
@pytest.mark.parametrize("layout", ["head_major", "token_major"])
def test_tiny_config_fused(rank_mode, layout):
    cfg = workloads.CONFIGS[0]
    lay = workloads.make_layer(cfg, 0, layout=layout)
    parity.run_fused_and_check(cfg, lay, rank_mode=rank_mode)


@pytest.mark.parametrize("scope", [binding.SCOPE_HEAD, binding.SCOPE_LAYER])
@pytest.mark.parametrize("rank_mode", [binding.RANK_POSITION, binding.RANK_SCORE])
@pytest.mark.parametrize("threshold", [0.01, 0.1])
def test_ragged_batch_fp32_all_modes(scope, rank_mode, threshold):
    # several tiles, ragged tails, a sequence shorter than the window, one of length 1
    cfg = small_cfg(num_q_heads=6, num_kv_heads=2, window=16, heavy_count=5)
    lay = workloads.make_layer(cfg, 0, seq_lens=[300, 129, 7, 1, 128, 1000])
    parity.run_fused_and_check(cfg, lay, rank_mode=rank_mode, scope=scope, threshold=threshold)


@pytest.mark.parametrize("dtype,d", [("bf16", 64), ("bf16", 128), ("fp32", 128)])
def test_generic_path_other_types_and_head_dims(dtype, d):
    cfg = small_cfg(dtype=dtype, head_dim=d, window=5, num_q_heads=3, num_kv_heads=1)
    lay = workloads.make_layer(cfg, 1, seq_lens=[257, 40])
    parity.run_fused_and_check(cfg, lay, rank_mode=binding.RANK_SCORE)
    parity.run_fused_and_check(cfg, lay, rank_mode=binding.RANK_POSITION, threshold=0.2)


def test_paper_default_single_query_row():
    cfg = small_cfg(window=1, num_q_heads=8, num_kv_heads=2, dtype="bf16", head_dim=128)
    lay = workloads.make_layer(cfg, 0, seq_lens=[777, 64])
    res, ref, _, _ = parity.run_fused_and_check(cfg, lay)
    # w = 1: every head's scores are one softmax row, so they sum to 1
    sums = res.scores.double().cpu().numpy()[:, :777].sum(axis=1)
    np.testing.assert_allclose(sums, 1.0, rtol=1e-4)


def test_flags_force_full_keep_window_and_nullable_outputs():
    cfg = small_cfg(window=8)
    lay = workloads.make_layer(cfg, 0, seq_lens=[200, 31])
    res, _, _, _ = parity.run_fused_and_check(cfg, lay, force_full=1)
    assert res.lengths.cpu().tolist() == [[200, 200], [31, 31]]
    parity.run_fused_and_check(cfg, lay, keep_window=0, threshold=0.5)
    parity.run_fused_and_check(cfg, lay, keep_window=0, threshold=0.5, rank_mode=binding.RANK_SCORE)
    parity.run_fused_and_check(cfg, lay, threshold=0.0)
    # scores and kept_idx may be left out: budgets and rows must not change
    p = binding.params_for(cfg, lay, rank_mode=binding.RANK_SCORE)
    args = [t.to(DEV) for t in (lay.q_win, lay.k, lay.v, lay.seq_start, lay.seq_len)]
    full = binding.compress_layer(p, *args, lay.total_tokens)
    bare = binding.compress_layer(p, *args, lay.total_tokens, want_scores=False, want_kept_idx=False)
    torch.cuda.synchronize()
    assert torch.equal(full.lengths, bare.lengths) and torch.equal(full.offsets, bare.offsets)
    rows = int(full.offsets[-1])
    assert torch.equal(parity.bits(full.k_out[:rows]), parity.bits(bare.k_out[:rows]))
    assert torch.equal(parity.bits(full.v_out[:rows]), parity.bits(bare.v_out[:rows]))


# ----------------------------------------------------------- single stages ----
def _device_inputs(lay):
    return [t.to(DEV) for t in (lay.q_win, lay.k, lay.v, lay.seq_start, lay.seq_len)]


def test_score_stage_alone():
    cfg = small_cfg(window=32)
    lay = workloads.make_layer(cfg, 0, seq_lens=[512, 100])
    p = binding.params_for(cfg, lay)
    q, k, v, ss, sl = _device_inputs(lay)
    total = lay.total_tokens
    ws = torch.empty(binding.refree_workspace_size(p, total), dtype=torch.uint8, device=DEV)
    scores = torch.full((p.num_kv_heads, total), float("nan"), device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.refree_score(p, q, k, ss, sl, total, scores, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    want = orc.score(parity.oracle_params(p), lay.q_win, lay.k, lay.seq_start, lay.seq_len)
    parity.check_scores(scores, want)


@pytest.mark.parametrize("rank_mode", [binding.RANK_POSITION, binding.RANK_SCORE])
@pytest.mark.parametrize("scope", [binding.SCOPE_HEAD, binding.SCOPE_LAYER])
def test_select_stage_fed_oracle_scores_is_exact(rank_mode, scope):
    """Same fp32 scores on both sides: budgets and kept sets must be identical
    (units whose oracle decision sits within 1e-9 of a tie are the only exception)."""
    cfg = small_cfg(window=16, num_kv_heads=2, num_q_heads=2)
    lens = [700, 5, 2100, 33]
    lay = workloads.make_layer(cfg, 0, seq_lens=lens)
    p = binding.params_for(cfg, lay, rank_mode=rank_mode, scope=scope)
    op = parity.oracle_params(p)
    sc32 = orc.score(op, lay.q_win, lay.k, lay.seq_start, lay.seq_len).astype(np.float32)
    sel = orc.select(op, sc32, lens)
    total = lay.total_tokens
    units = p.num_seqs * p.num_kv_heads
    ws = torch.empty(binding.refree_workspace_size(p, total), dtype=torch.uint8, device=DEV)
    lengths = torch.zeros(units, dtype=torch.int32, device=DEV)
    offsets = torch.zeros(units + 1, dtype=torch.int64, device=DEV)
    cap = p.num_kv_heads * total
    kept = torch.full((cap,), -1, dtype=torch.int32, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.refree_select_budget(p, torch.from_numpy(sc32).to(DEV), lay.seq_len.to(DEV), total, lengths, offsets,
                                 kept, cap, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    ties = parity.check_selection(p, lens, lengths, offsets, kept, sel, sc32, tie_tol=1e-9)
    assert ties == 0 or (sel.gap < 1e-9).any()


@pytest.mark.parametrize("case", ["uniform", "all_ties_score_mode", "zeros", "one_hot"])
def test_select_stage_closed_forms_on_device(case):
    n = 8192
    p = binding.Params(1, 1, 1, 128, window=1, sink=4, keep_window=0,
                       rank_mode=binding.RANK_SCORE if case == "all_ties_score_mode" else binding.RANK_POSITION)
    sc = np.full((1, n), 0.25, dtype=np.float32)
    want = 8029                       # floor((1 - T)^2 n) + 1
    if case == "zeros":
        sc[:] = 0.0
        want = n
    if case == "one_hot":
        sc[:] = 0.0
        sc[0, n - 10] = 1.0           # rank m + 10 in the position order
        want = 14
    ws = torch.empty(binding.refree_workspace_size(p, n), dtype=torch.uint8, device=DEV)
    lengths = torch.zeros(1, dtype=torch.int32, device=DEV)
    offsets = torch.zeros(2, dtype=torch.int64, device=DEV)
    kept = torch.zeros(n, dtype=torch.int32, device=DEV)
    binding.refree_select_budget(p, torch.from_numpy(sc).to(DEV), torch.tensor([n], dtype=torch.int32, device=DEV),
                                 n, lengths, offsets, kept, n, ws, None)
    torch.cuda.synchronize()
    assert lengths.item() == want
    sel = orc.select(parity.oracle_params(p), sc, [n])
    assert sel.lengths[0, 0] == want
    np.testing.assert_array_equal(kept[:want].cpu().numpy(), sel.kept_idx)


def test_compact_stage_fed_oracle_indices():
    cfg = small_cfg(window=8, dtype="bf16", head_dim=128)
    lay = workloads.make_layer(cfg, 0, seq_lens=[300, 77], layout="token_major")
    p = binding.params_for(cfg, lay, rank_mode=binding.RANK_SCORE)
    ref = orc.compress_layer(parity.oracle_params(p), lay.q_win, lay.k, lay.v, lay.seq_start, lay.seq_len)
    q, k, v, ss, sl = _device_inputs(lay)
    rows = int(ref.sel.offsets[-1])
    k_out = torch.zeros(rows, p.head_dim, dtype=k.dtype, device=DEV)
    v_out = torch.zeros_like(k_out)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.refree_compact(p, k, v, ss, sl, torch.from_numpy(ref.sel.lengths.reshape(-1)).to(DEV),
                           torch.from_numpy(ref.sel.offsets).to(DEV), torch.from_numpy(ref.sel.kept_idx).to(DEV),
                           k_out, v_out, rows, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    assert torch.equal(parity.bits(k_out.cpu()), parity.bits(ref.k_out))
    assert torch.equal(parity.bits(v_out.cpu()), parity.bits(ref.v_out))


# ---------------------------------------------------------------- errors ----
def test_capacity_overflow_is_reported_and_nothing_is_written_past_capacity():
    cfg = small_cfg(window=8)
    lay = workloads.make_layer(cfg, 0, seq_lens=[256])
    p = binding.params_for(cfg, lay, force_full=1)
    args = _device_inputs(lay)
    cap = 300                                     # needs 512
    k_out = torch.full((cap + 64, p.head_dim), 7.0, device=DEV)
    v_out = torch.full((cap + 64, p.head_dim), 7.0, device=DEV)
    lengths = torch.zeros(2, dtype=torch.int32, device=DEV)
    offsets = torch.zeros(3, dtype=torch.int64, device=DEV)
    ws = torch.empty(binding.refree_workspace_size(p, 256), dtype=torch.uint8, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.refree_compress_layer(p, *args, 256, k_out, v_out, cap, lengths, offsets, None, None, ws, st)
    torch.cuda.synchronize()
    assert st.item() & binding.DEV_CAPACITY
    assert (k_out[cap:] == 7.0).all() and (v_out[cap:] == 7.0).all()
    assert lengths.cpu().tolist() == [256, 256]


def test_host_buffer_entry_point_matches_device_entry_point():
    cfg = small_cfg(window=16)
    lay = workloads.make_layer(cfg, 0, seq_lens=[400, 90])
    p = binding.params_for(cfg, lay, rank_mode=binding.RANK_SCORE)
    total = lay.total_tokens
    cap = p.num_kv_heads * total
    dev_res = binding.compress_layer(p, *_device_inputs(lay), total)
    torch.cuda.synchronize()
    arena = torch.empty(binding.refree_host_arena_size(p, total, lay.k.numel(), cap), dtype=torch.uint8, device=DEV)
    k_out = torch.zeros(cap, p.head_dim, dtype=lay.k.dtype).pin_memory()
    v_out = torch.zeros(cap, p.head_dim, dtype=lay.k.dtype).pin_memory()
    units = p.num_seqs * p.num_kv_heads
    lengths = torch.zeros(units, dtype=torch.int32)
    offsets = torch.zeros(units + 1, dtype=torch.int64)
    kept = torch.zeros(cap, dtype=torch.int32)
    scores = torch.zeros(p.num_kv_heads, total)
    binding.refree_compress_layer_host(p, lay.q_win, lay.k, lay.v, lay.seq_start, lay.seq_len, total, k_out, v_out,
                                       cap, lengths, offsets, kept, scores, arena)
    rows = int(offsets[-1])
    assert torch.equal(lengths, dev_res.lengths.cpu().reshape(-1)) and torch.equal(offsets, dev_res.offsets.cpu())
    assert torch.equal(kept[:rows], dev_res.kept_idx[:rows].cpu())
    assert torch.equal(parity.bits(k_out[:rows]), parity.bits(dev_res.k_out[:rows].cpu()))
    assert torch.equal(parity.bits(v_out[:rows]), parity.bits(dev_res.v_out[:rows].cpu()))
    assert torch.equal(scores, dev_res.scores.cpu())


@pytest.mark.parametrize("rank_mode", [binding.RANK_POSITION, binding.RANK_SCORE])
@pytest.mark.parametrize("pinned", [True, False])
def test_pipelined_host_run_of_layers_matches_the_per_layer_call(rank_mode, pinned):
    # five layers through the three-stream pipeline (two staging slots, so slots are reused twice)
    cfg = small_cfg(window=16, dtype="bf16", head_dim=128, num_q_heads=8, num_kv_heads=2)
    n_layers = 5
    lays = [workloads.make_layer(cfg, l, seq_lens=[700, 90, 333]) for l in range(n_layers)]
    p = binding.params_for(cfg, lays[0], rank_mode=rank_mode, threshold=0.05)
    total = lays[0].total_tokens
    cap = p.num_kv_heads * total
    units = p.num_seqs * p.num_kv_heads
    pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    q = [pin(l.q_win) for l in lays]
    k = [pin(l.k) for l in lays]
    v = [pin(l.v) for l in lays]
    k_out = [pin(torch.zeros(cap, p.head_dim, dtype=lays[0].k.dtype)) for _ in lays]
    v_out = [pin(torch.zeros(cap, p.head_dim, dtype=lays[0].k.dtype)) for _ in lays]
    lengths = [torch.zeros(units, dtype=torch.int32) for _ in lays]
    offsets = [torch.zeros(units + 1, dtype=torch.int64) for _ in lays]
    arena = torch.empty(binding.refree_host_pipeline_arena_size(p, total, lays[0].k.numel(), cap), dtype=torch.uint8,
                        device=DEV)
    binding.refree_compress_layers_host(p, q, k, v, lays[0].seq_start, lays[0].seq_len, total, k_out, v_out, cap,
                                        lengths, offsets, arena)
    for l, lay in enumerate(lays):
        ref = binding.compress_layer(p, *_device_inputs(lay), total, want_scores=False, want_kept_idx=False)
        torch.cuda.synchronize()
        rows = int(offsets[l][-1])
        assert torch.equal(lengths[l], ref.lengths.cpu().reshape(-1)) and torch.equal(offsets[l], ref.offsets.cpu())
        assert torch.equal(parity.bits(k_out[l][:rows]), parity.bits(ref.k_out[:rows].cpu()))
        assert torch.equal(parity.bits(v_out[l][:rows]), parity.bits(ref.v_out[:rows].cpu()))


@pytest.mark.parametrize("rank_mode,window,dtype", [(binding.RANK_POSITION, 16, "bf16"), (binding.RANK_SCORE, 16, "bf16"),
                                                    (binding.RANK_POSITION, 1, "bf16"), (binding.RANK_POSITION, 8, "fp32"),
                                                    (binding.RANK_POSITION, 300, "bf16")])    # 1200 query rows: scored in chunks
def test_pipelined_device_run_of_layers_matches_the_per_layer_call(rank_mode, window, dtype):
    """refree_compress_layers (scoring of layer l + 1 over the compaction of layer l, two internal
    streams, two workspace halves) against one refree_compress_layer call per layer: five layers, so
    each half is reused, twice in a row on the same buffers, then once more after other work on the
    caller's stream."""
    cfg = small_cfg(window=window, dtype=dtype, head_dim=128, num_q_heads=8, num_kv_heads=2)
    n_layers = 5
    lays = [workloads.make_layer(cfg, l, seq_lens=[2700, 0, 90, 1333, 1]) for l in range(n_layers)]
    p = binding.params_for(cfg, lays[0], rank_mode=rank_mode, threshold=0.05)
    total = lays[0].total_tokens
    cap = p.num_kv_heads * total
    units = p.num_seqs * p.num_kv_heads
    dev_in = [_device_inputs(l) for l in lays]
    refs = [binding.compress_layer(p, *d, total, want_scores=False, want_kept_idx=False) for d in dev_in]
    torch.cuda.synchronize()
    k_out = [torch.zeros(cap, p.head_dim, dtype=lays[0].k.dtype, device=DEV) for _ in lays]
    v_out = [torch.zeros(cap, p.head_dim, dtype=lays[0].k.dtype, device=DEV) for _ in lays]
    lengths = [torch.zeros(units, dtype=torch.int32, device=DEV) for _ in lays]
    offsets = [torch.zeros(units + 1, dtype=torch.int64, device=DEV) for _ in lays]
    ptrs = binding.LayerPointers([d[0] for d in dev_in], [d[1] for d in dev_in], [d[2] for d in dev_in], k_out, v_out,
                                 lengths, offsets)
    ws = torch.empty(binding.refree_layers_workspace_size(p, total), dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    for rep in range(3):
        for t in k_out + v_out + lengths + offsets:
            t.fill_(0 if rep != 1 else 1)              # ordered before the run on the caller's stream
        binding.refree_compress_layers(p, ptrs, dev_in[0][3], dev_in[0][4], total, cap, ws, status)
        got = [(ln.clone(), of.clone(), ko.clone(), vo.clone()) for ln, of, ko, vo in zip(lengths, offsets, k_out, v_out)]
        torch.cuda.synchronize()                       # the clones were ordered after the run by the join
        assert status.item() == 0
        for l, ref in enumerate(refs):
            ln, of, ko, vo = got[l]
            rows = int(of[-1])
            assert rows == int(ref.offsets[-1]) and 0 < rows <= cap
            assert torch.equal(ln, ref.lengths.reshape(-1)) and torch.equal(of, ref.offsets)
            assert torch.equal(parity.bits(ko[:rows]), parity.bits(ref.k_out[:rows]))
            assert torch.equal(parity.bits(vo[:rows]), parity.bits(ref.v_out[:rows]))


def test_pipelined_device_run_rejects_a_single_workspace():
    cfg = small_cfg(window=16, dtype="bf16", head_dim=128, num_q_heads=8, num_kv_heads=2)
    lay = workloads.make_layer(cfg, 0, seq_lens=[300])
    p = binding.params_for(cfg, lay)
    d = _device_inputs(lay)
    cap = p.num_kv_heads * 300
    outs = [torch.zeros(cap, 128, dtype=lay.k.dtype, device=DEV) for _ in range(2)]
    ln, of = torch.zeros(2, dtype=torch.int32, device=DEV), torch.zeros(3, dtype=torch.int64, device=DEV)
    ptrs = binding.LayerPointers([d[0]], [d[1]], [d[2]], [outs[0]], [outs[1]], [ln], [of])
    ws = torch.empty(binding.refree_workspace_size(p, 300), dtype=torch.uint8, device=DEV)
    assert binding.refree_compress_layers(p, ptrs, d[3], d[4], 300, cap, ws, check=False) == binding.ERR_WORKSPACE


@pytest.mark.parametrize("dtype,d,hq,hkv", [("bf16", 128, 28, 4), ("fp32", 64, 4, 2), ("bf16", 64, 16, 1), ("fp32", 128, 3, 3)])
@pytest.mark.parametrize("rank_mode,scope", [(binding.RANK_POSITION, binding.SCOPE_HEAD),
                                             (binding.RANK_SCORE, binding.SCOPE_HEAD),
                                             (binding.RANK_POSITION, binding.SCOPE_LAYER)])
def test_single_query_row_path_shapes_and_modes(dtype, d, hq, hkv, rank_mode, scope):
    """w = 1 (the paper's default) has a scoring path of its own: group sizes 1..16,
    both storage types and head dims, ragged lengths down to one token."""
    cfg = small_cfg(window=1, num_q_heads=hq, num_kv_heads=hkv, dtype=dtype, head_dim=d)
    lay = workloads.make_layer(cfg, 2, seq_lens=[1, 300, 257, 4000, 31])
    parity.run_fused_and_check(cfg, lay, rank_mode=rank_mode, scope=scope)
