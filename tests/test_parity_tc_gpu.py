"""GPU parity of the tensor-core scoring path (bf16, head_dim 128) and of the
fused pass on bf16 caches, against the CPU oracle."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import refree_oracle as orc
from paper_2502_16886_b200 import binding, build, workloads
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
BASE = workloads.CONFIGS[1]          # 32 q / 8 kv heads, d 128, bf16, window 64


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def cfg_with(**kw):
    return dataclasses.replace(BASE, num_layers=1, **kw)


@pytest.mark.parametrize("hq,hkv,w,lens", [
    (8, 2, 64, [1000]),                    # 256 rows, several tiles and a ragged tail
    (8, 2, 64, [128, 129, 64, 65, 700]),   # tile-aligned, one over, exactly the window, window + 1
    (7, 1, 64, [900, 300]),                # 448 rows (GQA 7): two accumulators per tile
    (16, 2, 64, [520]),                    # 512 rows (GQA 8)
    (4, 2, 16, [400, 50]),                 # 32 rows: one partly filled row block
    (8, 2, 64, [40, 1, 300]),              # sequences shorter than the window
])
def test_tc_scores_match_oracle(hq, hkv, w, lens):
    cfg = cfg_with(num_q_heads=hq, num_kv_heads=hkv, window=w)
    lay = workloads.make_layer(cfg, 0, seq_lens=lens)
    p = binding.params_for(cfg, lay)
    q, k, ss, sl = [t.to(DEV) for t in (lay.q_win, lay.k, lay.seq_start, lay.seq_len)]
    total = lay.total_tokens
    ws = torch.empty(binding.refree_workspace_size(p, total), dtype=torch.uint8, device=DEV)
    scores = torch.full((hkv, total), float("nan"), device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.refree_score(p, q, k, ss, sl, total, scores, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    want = orc.score(parity.oracle_params(p), lay.q_win, lay.k, lay.seq_start, lay.seq_len)
    worst = parity.check_scores(scores, want)
    assert worst < 1e-4          # fp32 softmax of exact bf16 products: far inside the 1e-3 bar


@pytest.mark.parametrize("layout", ["head_major", "token_major"])
@pytest.mark.parametrize("rank_mode", [binding.RANK_POSITION, binding.RANK_SCORE])
def test_tc_fused_pass_both_layouts(layout, rank_mode):
    cfg = cfg_with(num_q_heads=8, num_kv_heads=2)
    lay = workloads.make_layer(cfg, 3, layout=layout, seq_lens=[2000, 333])
    parity.run_fused_and_check(cfg, lay, rank_mode=rank_mode)


def test_tc_padded_batch_layout_with_sequence_stride():
    """[B, Hkv, n_max, d] cache with per-sequence lengths below n_max: the token
    axis restarts at 0 for every sequence and a sequence stride is in play."""
    cfg = cfg_with(num_q_heads=8, num_kv_heads=2)
    lens, n_max = [300, 517, 64], 640
    lay = workloads.make_layer(cfg, 0, seq_lens=lens)
    B, Hkv, d = len(lens), 2, 128
    kp = torch.zeros(B, Hkv, n_max, d, dtype=torch.bfloat16)
    vp = torch.zeros(B, Hkv, n_max, d, dtype=torch.bfloat16)
    for s, n in enumerate(lens):
        a = int(lay.seq_start[s])
        kp[s, :, :n] = lay.k[:, a:a + n]
        vp[s, :, :n] = lay.v[:, a:a + n]
    strides = (Hkv * n_max * d, d, n_max * d)
    p = binding.params_for(cfg, lay, kv_tokens=n_max, k_strides=strides, v_strides=strides)
    zero = torch.zeros(B, dtype=torch.int32)
    total = sum(lens)
    res = binding.compress_layer(p, lay.q_win.to(DEV), kp.to(DEV), vp.to(DEV), zero.to(DEV), lay.seq_len.to(DEV), total)
    torch.cuda.synchronize()
    assert res.device_status.item() == 0
    ref = orc.compress_layer(parity.oracle_params(p), lay.q_win, kp, vp, zero, lay.seq_len)
    parity.check_scores(res.scores, ref.scores)
    parity.check_selection(p, lens, res.lengths, res.offsets, res.kept_idx, ref.sel, ref.scores32)
    rows = int(ref.sel.offsets[-1])
    if torch.equal(res.lengths.cpu().reshape(-1), torch.from_numpy(ref.sel.lengths.reshape(-1))):
        assert torch.equal(parity.bits(res.k_out[:rows].cpu()), parity.bits(ref.k_out))
        assert torch.equal(parity.bits(res.v_out[:rows].cpu()), parity.bits(ref.v_out))


def test_tc_large_logits_do_not_overflow():
    """Keys scaled so that logits reach the hundreds: the running reference of
    pass 1 must be refreshed when a later tile dwarfs the first one."""
    cfg = cfg_with(num_q_heads=8, num_kv_heads=2)
    lay = workloads.make_layer(cfg, 1, seq_lens=[1500])
    lay.k[:, 700:710] *= 40.0          # a few late, very loud keys
    p = binding.params_for(cfg, lay)
    q, k, ss, sl = [t.to(DEV) for t in (lay.q_win, lay.k, lay.seq_start, lay.seq_len)]
    ws = torch.empty(binding.refree_workspace_size(p, 1500), dtype=torch.uint8, device=DEV)
    scores = torch.empty(2, 1500, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.refree_score(p, q, k, ss, sl, 1500, scores, ws, st)
    torch.cuda.synchronize()
    assert st.item() == 0
    want = orc.score(parity.oracle_params(p), lay.q_win, lay.k, lay.seq_start, lay.seq_len)
    parity.check_scores(scores, want)
