"""Paged compaction (refree_compact_paged) against the oracle.

The oracle selects and compacts on the CPU (dense ragged ``K_c, V_c``); the kernel
is given the oracle's selection and a shuffled block table, and every block of the
pools must hold, bit for bit, the rows of the oracle's dense output that the
table assigns to it.  Blocks the budgets do not reach stay untouched.
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


def _setup(cfg, lay, p, block_rows, seed):
    rng = np.random.default_rng(seed)
    scores = (rng.random((p.num_kv_heads, lay.total_tokens)) ** 4).astype(np.float32)
    op = parity.oracle_params(p)
    sel = orc.select(op, scores, lay.seq_len)
    want_k, want_v = orc.compact(op, lay.k, lay.v, lay.seq_start, lay.seq_len, sel)
    units = p.num_seqs * p.num_kv_heads
    per_unit = [-(-int(lay.seq_len[u // p.num_kv_heads]) // block_rows) for u in range(units)]   # worst case: keep all
    max_blocks = max(1, max(per_unit))
    num_blocks = sum(per_unit) + 3
    order = rng.permutation(num_blocks)
    table = np.full((units, max_blocks), -1, dtype=np.int32)
    nxt = 0
    for u in range(units):
        table[u, :per_unit[u]] = order[nxt:nxt + per_unit[u]]
        nxt += per_unit[u]
    return sel, want_k, want_v, table, num_blocks


@pytest.mark.parametrize("rank_mode", [binding.RANK_POSITION, binding.RANK_SCORE])
@pytest.mark.parametrize("layout,dtype,d,block_rows", [("head_major", "bf16", 128, 16), ("token_major", "bf16", 128, 256),
                                                       ("head_major", "fp32", 64, 7), ("token_major", "fp32", 128, 32)])
def test_paged_compaction_matches_the_oracle(rank_mode, layout, dtype, d, block_rows):
    cfg = _cfg(window=16, dtype=dtype, head_dim=d, num_q_heads=6, num_kv_heads=3)
    lay = workloads.make_layer(cfg, 1, layout=layout, seq_lens=[9000, 90, 0, 4001, 1, 16])
    p = binding.params_for(cfg, lay, rank_mode=rank_mode, threshold=0.1)
    sel, want_k, want_v, table, num_blocks = _setup(cfg, lay, p, block_rows, seed=3)
    fill = 7.0
    k_pool = torch.full((num_blocks, block_rows, d), fill, dtype=lay.k.dtype, device=DEV)
    v_pool = torch.full((num_blocks, block_rows, d), fill, dtype=lay.k.dtype, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ranges = rank_mode == binding.RANK_POSITION
    kept = torch.from_numpy(sel.kept_idx if sel.kept_idx.size else np.zeros(1, np.int32)).to(DEV)
    binding.refree_compact_paged(p, lay.k.to(DEV), lay.v.to(DEV), lay.seq_start.to(DEV), lay.seq_len.to(DEV),
                                 torch.from_numpy(sel.lengths.reshape(-1).copy()).to(DEV),
                                 None if ranges else torch.from_numpy(sel.offsets).to(DEV), None if ranges else kept,
                                 torch.from_numpy(table).to(DEV), block_rows, k_pool, v_pool, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    k_pool, v_pool = k_pool.cpu(), v_pool.cpu()
    untouched = torch.full((block_rows, d), fill, dtype=lay.k.dtype)
    used = set()
    for u in range(table.shape[0]):
        a, b = int(sel.offsets[u]), int(sel.offsets[u + 1])
        for j in range(table.shape[1]):
            blk = int(table[u, j])
            if blk < 0:
                continue
            used.add(blk)
            rows = max(0, min(block_rows, (b - a) - j * block_rows))
            lo = a + j * block_rows
            assert torch.equal(parity.bits(k_pool[blk, :rows]), parity.bits(want_k[lo:lo + rows]))
            assert torch.equal(parity.bits(v_pool[blk, :rows]), parity.bits(want_v[lo:lo + rows]))
            assert torch.equal(k_pool[blk, rows:], untouched[rows:]) and torch.equal(v_pool[blk, rows:], untouched[rows:])
    for blk in set(range(num_blocks)) - used:
        assert torch.equal(k_pool[blk], untouched) and torch.equal(v_pool[blk], untouched)
    assert 0 < int(sel.offsets[-1]) < p.num_kv_heads * lay.total_tokens


def test_paged_compaction_flags_a_table_that_is_too_short_or_out_of_range():
    cfg = _cfg(window=8, dtype="bf16", head_dim=128, num_q_heads=2, num_kv_heads=1)
    lay = workloads.make_layer(cfg, 0, seq_lens=[100])
    p = binding.params_for(cfg, lay, force_full=1)
    k, v, ss, sl = [t.to(DEV) for t in (lay.k, lay.v, lay.seq_start, lay.seq_len)]
    lengths = torch.tensor([100], dtype=torch.int32, device=DEV)
    k_pool = torch.zeros(5, 16, 128, dtype=lay.k.dtype, device=DEV)
    v_pool = torch.zeros_like(k_pool)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    short = torch.tensor([[0, 1, 2, 3]], dtype=torch.int32, device=DEV)            # 64 rows of room for 100
    binding.refree_compact_paged(p, k, v, ss, sl, lengths, None, None, short, 16, k_pool, v_pool, status)
    torch.cuda.synchronize()
    assert status.item() & binding.DEV_CAPACITY and not k_pool.any()
    status.zero_()
    wild = torch.tensor([[0, 1, 2, 3, 9, -1, 4]], dtype=torch.int32, device=DEV)     # blocks 9 and -1 do not exist
    binding.refree_compact_paged(p, k, v, ss, sl, lengths, None, None, wild, 16, k_pool, v_pool, status)
    torch.cuda.synchronize()
    assert status.item() & binding.DEV_CAPACITY
    assert torch.equal(parity.bits(k_pool[0].cpu()), parity.bits(lay.k[0, :16]))     # the valid blocks were written
