"""Edge cases of the pass on the GPU, each through every scoring path (tensor-core,
single query row, generic) and both rankings: empty sequences inside a batch, the
largest row counts each path takes, and score ranking when a cluster of blocks
shares a unit whose sequences are far shorter than the batch mean."""
import dataclasses

import pytest
import torch

from paper_2502_16886_b200 import binding, build, workloads
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def cfg_like(**kw):
    return dataclasses.replace(workloads.CONFIGS[0], **kw)


@pytest.mark.parametrize("rank_mode", [binding.RANK_POSITION, binding.RANK_SCORE])
@pytest.mark.parametrize("path", ["generic_fp32", "tensor_core", "single_row"])
def test_empty_sequences_inside_a_batch(path, rank_mode):
    if path == "generic_fp32":
        cfg = cfg_like(num_q_heads=4, num_kv_heads=2, window=8)
    elif path == "tensor_core":
        cfg = cfg_like(dtype="bf16", head_dim=128, num_q_heads=8, num_kv_heads=2, window=16)
    else:
        cfg = cfg_like(dtype="bf16", head_dim=128, num_q_heads=8, num_kv_heads=2, window=1)
    lay = workloads.make_layer(cfg, 0, seq_lens=[0, 300, 0, 0, 5, 129, 0])
    res, ref, _, _ = parity.run_fused_and_check(cfg, lay, rank_mode=rank_mode)
    lengths = res.lengths.cpu()
    assert (lengths[[0, 2, 3, 6]] == 0).all()           # an empty sequence keeps nothing
    assert (lengths[[1, 4, 5]] >= 1).all()


def test_batch_of_only_empty_sequences():
    # the cache buffers exist (16 rows) but every sequence is empty: nothing kept, nothing written
    dev = torch.device("cuda:0")
    hq, hkv, d, w, rows = 4, 2, 64, 8, 16
    p = binding.Params(num_seqs=2, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, window=w, dtype=binding.DTYPE_F32,
                       kv_tokens=rows, k_strides=(0, d, rows * d), v_strides=(0, d, rows * d))
    k = torch.randn(hkv, rows, d, device=dev)
    v = torch.randn(hkv, rows, d, device=dev)
    q = torch.randn(2, hq, w, d, device=dev)
    zeros = torch.zeros(2, dtype=torch.int32, device=dev)
    res = binding.compress_layer(p, q, k, v, zeros, zeros, 0, capacity_rows=4)
    torch.cuda.synchronize()
    assert int(res.device_status.item()) == 0
    assert (res.lengths == 0).all() and (res.offsets == 0).all()


@pytest.mark.parametrize("hq,hkv,w", [(8, 1, 64), (16, 2, 64), (4, 1, 128)])
def test_largest_row_count_of_the_tensor_core_path(hq, hkv, w):
    # G * w = 512 rows: four row blocks in pass 1, four column blocks in pass 2
    cfg = cfg_like(dtype="bf16", head_dim=128, num_q_heads=hq, num_kv_heads=hkv, window=w)
    lay = workloads.make_layer(cfg, 0, seq_lens=[1000, 77])
    parity.run_fused_and_check(cfg, lay)
    parity.run_fused_and_check(cfg, lay, rank_mode=binding.RANK_SCORE)


def test_largest_row_count_of_the_generic_path():
    # G * w = 1024 rows, fp32
    cfg = cfg_like(num_q_heads=8, num_kv_heads=1, window=128)
    lay = workloads.make_layer(cfg, 0, seq_lens=[400, 130])
    parity.run_fused_and_check(cfg, lay)


def test_sixteen_query_heads_per_kv_head_single_row():
    cfg = cfg_like(dtype="bf16", head_dim=128, num_q_heads=32, num_kv_heads=2, window=1)
    lay = workloads.make_layer(cfg, 0, seq_lens=[2000, 33])
    parity.run_fused_and_check(cfg, lay)


@pytest.mark.parametrize("scope", [binding.SCOPE_HEAD, binding.SCOPE_LAYER])
@pytest.mark.parametrize("threshold", [0.01, 0.2])
def test_score_ranking_with_a_cluster_per_unit_on_a_ragged_batch(scope, threshold):
    # the mean length (about 10 K) puts two blocks on every unit, also on the sequences of 1, 40 and
    # 300 positions, where all but one block of the cluster have no positions at all
    cfg = cfg_like(dtype="bf16", head_dim=128, num_q_heads=8, num_kv_heads=2, window=16, heavy_count=40)
    lay = workloads.make_layer(cfg, 0, seq_lens=[30000, 300, 1, 20000, 40])
    parity.run_fused_and_check(cfg, lay, rank_mode=binding.RANK_SCORE, scope=scope, threshold=threshold)


def test_score_ranking_with_eight_blocks_per_unit():
    cfg = cfg_like(dtype="bf16", head_dim=128, num_q_heads=4, num_kv_heads=1, window=32, heavy_count=200)
    lay = workloads.make_layer(cfg, 0, seq_lens=[40000])
    parity.run_fused_and_check(cfg, lay, rank_mode=binding.RANK_SCORE)
    parity.run_fused_and_check(cfg, lay, rank_mode=binding.RANK_SCORE, scope=binding.SCOPE_LAYER, threshold=0.05)


def test_score_ranking_with_units_on_both_sides_of_what_a_cluster_holds_in_registers():
    # score ranking per head keeps a unit's keys in the registers of a cluster of blocks when they fit
    # (8 blocks x 1024 threads x 16 keys); here one sequence is longer than that and goes to the kernel
    # that re-reads the scores, the others do not, and the index list is written for both kinds in one launch
    cfg = cfg_like(dtype="bf16", head_dim=128, num_q_heads=2, num_kv_heads=1, window=16, heavy_count=300)
    lay = workloads.make_layer(cfg, 0, seq_lens=[140_000, 700, 9000])
    parity.run_fused_and_check(cfg, lay, rank_mode=binding.RANK_SCORE)


@pytest.mark.parametrize("n", [1023, 1024, 1025, 4096, 20_000])
def test_score_ranking_with_many_equal_scores_at_the_crossing(n):
    # equal scores at the crossing key: the lowest positions among them are kept, whatever run of 1024
    # positions (one block of the kernel that writes the index list) they fall into
    cfg = cfg_like(num_q_heads=2, num_kv_heads=1, window=4)
    p = binding.Params(num_seqs=1, num_q_heads=2, num_kv_heads=1, head_dim=64, window=4, sink=2, threshold=0.3,
                       rank_mode=binding.RANK_SCORE, dtype=binding.DTYPE_F32, kv_tokens=n,
                       k_strides=(0, 64, n * 64), v_strides=(0, 64, n * 64))
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(n)
    vals = torch.tensor([0.5, 0.25, 0.125, 0.0625])
    scores = vals[torch.randint(0, 4, (1, n), generator=g)].contiguous()
    sl = torch.tensor([n], dtype=torch.int32)
    lengths = torch.zeros(1, dtype=torch.int32, device=dev)
    offsets = torch.zeros(2, dtype=torch.int64, device=dev)
    kept = torch.full((n,), -1, dtype=torch.int32, device=dev)
    ws = torch.empty(binding.refree_workspace_size(p, n), dtype=torch.uint8, device=dev)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    binding.refree_select_budget(p, scores.to(dev), sl.to(dev), n, lengths, offsets, kept, n, ws, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    b = int(lengths.item())
    got = kept[:b].cpu().tolist()
    # brute force: protected positions first, then by decreasing score, ties by position
    a = scores[0].double().numpy()
    prot = [0, 1] + list(range(n - 4, n))
    rest = sorted((i for i in range(2, n - 4)), key=lambda i: (-a[i], i))
    order = prot + rest
    import numpy as np
    c = np.cumsum(a[order] ** 2)
    j = int(np.argmax(1.0 - np.sqrt(c / c[-1]) < 0.3)) + 1
    want_b = max(j, len(prot))
    assert b == want_b
    assert got == sorted(order[:b])


def test_position_ranking_beyond_the_length_the_record_fed_rule_takes():
    # above 131072 tokens in a call the budgets come from the rule that reads every score
    cfg = cfg_like(dtype="bf16", head_dim=128, num_q_heads=2, num_kv_heads=1, window=16, heavy_count=300)
    lay = workloads.make_layer(cfg, 0, seq_lens=[140_000, 700])
    parity.run_fused_and_check(cfg, lay)


@pytest.mark.parametrize("kind", ["tensor_core_chunks", "generic_chunks"])
@pytest.mark.parametrize("rank_mode", [binding.RANK_POSITION, binding.RANK_SCORE])
def test_windows_longer_than_one_scoring_pass_are_scored_in_chunks(kind, rank_mode):
    # Section 4.4 studies windows of up to a tenth of the sequence: G * w beyond 1024 query rows is scored in
    # chunks of window rows (512 rows on the tensor-core path, 1024 on the generic one), the last chunk ragged,
    # with one sequence shorter than the window and one shorter than a chunk
    if kind == "tensor_core_chunks":
        cfg = cfg_like(dtype="bf16", head_dim=128, num_q_heads=8, num_kv_heads=2, window=300, heavy_count=60)
    else:
        cfg = cfg_like(num_q_heads=4, num_kv_heads=2, window=1100, heavy_count=60)
    lay = workloads.make_layer(cfg, 0, seq_lens=[3000, 200, 0, 90])
    parity.run_fused_and_check(cfg, lay, rank_mode=rank_mode)


def test_rows_beyond_what_chunks_cover_are_refused():
    p = binding.Params(num_seqs=1, num_q_heads=4, num_kv_heads=1, head_dim=64, window=10_000, dtype=binding.DTYPE_F32,
                       kv_tokens=16, k_strides=(0, 64, 16 * 64), v_strides=(0, 64, 16 * 64))
    with pytest.raises(binding.RefreeError):
        binding.refree_workspace_size(p, 16)
