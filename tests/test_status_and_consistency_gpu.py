"""Device-status conditions made on the host (a bad index list, non-finite keys), none of which may
fault, and the agreement of the two arithmetics that implement the stopping rule on the GPU."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2502_16886_b200 import binding, build, workloads
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def test_compact_reports_an_index_outside_the_sequence_and_reads_nothing_there():
    cfg = dataclasses.replace(workloads.CONFIGS[1], num_layers=1, num_q_heads=8, num_kv_heads=2)
    lay = workloads.make_layer(cfg, 0, seq_lens=[300])
    p = binding.params_for(cfg, lay, rank_mode=binding.RANK_SCORE)
    n, hkv, d = 300, 2, cfg.head_dim
    k, v, ss, sl = [t.to(DEV) for t in (lay.k, lay.v, lay.seq_start, lay.seq_len)]
    lengths = torch.tensor([5, 4], dtype=torch.int32, device=DEV)
    offsets = torch.tensor([0, 5, 9], dtype=torch.int64, device=DEV)
    # unit 0: rows 3 and 4 of its list are out of range (beyond n, negative); unit 1 is clean
    kept = torch.tensor([0, 7, 9, n + 50_000, -3, 1, 2, 3, 299], dtype=torch.int32, device=DEV)
    fill = torch.full((9, d), 7.0, dtype=lay.k.dtype, device=DEV)
    k_out, v_out = fill.clone(), fill.clone()
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.refree_compact(p, k, v, ss, sl, lengths, offsets, kept, k_out, v_out, 9, st)
    torch.cuda.synchronize()
    assert int(st.item()) & binding.DEV_CAPACITY
    good = [0, 1, 2, 5, 6, 7, 8]
    src_unit = [0, 0, 0, 1, 1, 1, 1]
    for row, u in zip(good, src_unit):
        assert torch.equal(parity.bits(k_out[row]), parity.bits(k[u, int(kept[row])]))
        assert torch.equal(parity.bits(v_out[row]), parity.bits(v[u, int(kept[row])]))
    for row in (3, 4):                                   # rows with a bad source are left as they were
        assert torch.equal(k_out[row], fill[row]) and torch.equal(v_out[row], fill[row])


@pytest.mark.parametrize("bad", [float("nan"), float("inf")])
@pytest.mark.parametrize("window", [64, 1])
def test_non_finite_key_sets_the_status_bit_and_leaves_other_units_alone(bad, window):
    cfg = dataclasses.replace(workloads.CONFIGS[1], num_layers=1, num_q_heads=8, num_kv_heads=2, window=window)
    lay = workloads.make_layer(cfg, 1, seq_lens=[700, 400])
    p = binding.params_for(cfg, lay)
    q, ss, sl = [t.to(DEV) for t in (lay.q_win, lay.seq_start, lay.seq_len)]
    total = lay.total_tokens
    ws = torch.empty(binding.refree_workspace_size(p, total), dtype=torch.uint8, device=DEV)

    def run(k):
        scores = torch.zeros((2, total), device=DEV)
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        binding.refree_score(p, q, k.to(DEV), ss, sl, total, scores, ws, st)
        torch.cuda.synchronize()
        return scores.cpu(), int(st.item())

    clean, st0 = run(lay.k)
    assert st0 == 0
    k_bad = lay.k.clone()
    k_bad[1, 123, 5] = bad                                # head 1, position 123 of the first sequence
    dirty, st1 = run(k_bad)
    assert st1 & binding.DEV_NONFINITE and not st1 & binding.DEV_TIMEOUT
    # units that do not contain the bad key: head 0 everywhere, head 1 of the second sequence
    assert torch.equal(dirty[0], clean[0])
    assert torch.equal(dirty[1, 700:], clean[1, 700:])
    assert not torch.isfinite(dirty[1, :700]).all()


@pytest.mark.parametrize("name", ["mistral7b_32k", "qwen25_7b_ragged8", "llama3_8b_8k"])
def test_fused_budgets_equal_the_staged_selection_on_the_same_gpu_scores(name):
    """Position ranking per head has two implementations of one rule: the fused pass takes its budgets from
    per-32-position sums that the scoring kernel leaves, refree_select_budget sums every score itself.  Fed
    the same GPU scores they must agree exactly, at full size."""
    cfg = workloads.get_config(name)
    lay = workloads.make_layer(cfg, 0)
    p = binding.params_for(cfg, lay)
    total = lay.total_tokens
    res = binding.compress_layer(p, lay.q_win.to(DEV), lay.k.to(DEV), lay.v.to(DEV), lay.seq_start.to(DEV),
                                 lay.seq_len.to(DEV), total, want_scores=True, want_kept_idx=False)
    torch.cuda.synchronize()
    assert int(res.device_status.item()) == 0
    units = p.num_seqs * p.num_kv_heads
    lengths = torch.zeros(units, dtype=torch.int32, device=DEV)
    offsets = torch.zeros(units + 1, dtype=torch.int64, device=DEV)
    ws = torch.empty(binding.refree_workspace_size(p, total), dtype=torch.uint8, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.refree_select_budget(p, res.scores, lay.seq_len.to(DEV), total, lengths, offsets, None,
                                 p.num_kv_heads * total, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    np.testing.assert_array_equal(lengths.cpu().numpy(), res.lengths.reshape(-1).cpu().numpy())
    np.testing.assert_array_equal(offsets.cpu().numpy(), res.offsets.cpu().numpy())
    torch.cuda.empty_cache()


@pytest.mark.parametrize("bulk", [False, True])
def test_memory_probes_copy_the_rows_they_say(bulk):
    # the probes only exist to put a ceiling beside the benchmark's numbers, but what they move must be right
    rows, kept, d = 5000, 4321, 128
    k = torch.randn(rows, d, device=DEV).to(torch.bfloat16)
    v = torch.randn(rows, d, device=DEV).to(torch.bfloat16)
    k_out = torch.zeros(kept, d, dtype=torch.bfloat16, device=DEV)
    v_out = torch.zeros(kept, d, dtype=torch.bfloat16, device=DEV)
    binding.refree_sol_row_mix(k, v, k_out, v_out, rows, kept, d * 2, bulk=bulk)
    binding.refree_sol_read_stream(k, bulk=bulk)
    torch.cuda.synchronize()
    assert torch.equal(parity.bits(k_out), parity.bits(k[rows - kept:]))
    assert torch.equal(parity.bits(v_out), parity.bits(v[rows - kept:]))


def test_record_fed_rule_equals_the_rule_that_reads_every_score_at_its_longest_sequence():
    """131072 positions is the longest call whose budgets come from the per-32-position records; there its
    coarser fixed point must still give the budgets of the rule that reads every score."""
    cfg = dataclasses.replace(workloads.CONFIGS[1], num_layers=1, num_q_heads=4, num_kv_heads=2, window=16)
    lay = workloads.make_layer(cfg, 0, seq_lens=[131_072])
    p = binding.params_for(cfg, lay)
    total = lay.total_tokens
    res = binding.compress_layer(p, lay.q_win.to(DEV), lay.k.to(DEV), lay.v.to(DEV), lay.seq_start.to(DEV),
                                 lay.seq_len.to(DEV), total, want_scores=True, want_kept_idx=False)
    torch.cuda.synchronize()
    assert int(res.device_status.item()) == 0
    units = p.num_seqs * p.num_kv_heads
    lengths = torch.zeros(units, dtype=torch.int32, device=DEV)
    offsets = torch.zeros(units + 1, dtype=torch.int64, device=DEV)
    ws = torch.empty(binding.refree_workspace_size(p, total), dtype=torch.uint8, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.refree_select_budget(p, res.scores, lay.seq_len.to(DEV), total, lengths, offsets, None,
                                 p.num_kv_heads * total, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    np.testing.assert_array_equal(lengths.cpu().numpy(), res.lengths.reshape(-1).cpu().numpy())
