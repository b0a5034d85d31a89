"""The no-allocation selection entry point against the regular one.

Some users of this library cannot allocate device memory when they compress a
cache (a serving engine whose pool is fully committed, a plug-in whose host
forbids cudaMalloc after start-up).  ``refree_select_budget_static`` serves
them with a scratch array built into the library.  This test calls it through
the C ABI twice in a row, on different inputs, and requires the same budgets,
offsets and kept positions as ``refree_select_budget`` (integer outputs, so the
comparison is exact).  It lives in a file that sorts last so that a run which
stops at the first failure has already exercised everything else.
"""
import numpy as np
import pytest
import torch

from paper_2502_16886_b200 import binding, build

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run(entry, p, scores, seq_len, total, with_workspace):
    units = p.num_seqs * p.num_kv_heads
    cap = p.num_kv_heads * total
    lengths = torch.full((units,), -7, dtype=torch.int32, device=DEV)
    offsets = torch.full((units + 1,), -7, dtype=torch.int64, device=DEV)
    kept = torch.full((cap,), -7, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    if with_workspace:
        ws = torch.empty(binding.refree_workspace_size(p, total), dtype=torch.uint8, device=DEV)
        entry(p, scores, seq_len, total, lengths, offsets, kept, cap, ws, status)
    else:
        entry(p, scores, seq_len, total, lengths, offsets, kept, cap, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    return lengths.cpu(), offsets.cpu(), kept.cpu()


@pytest.mark.parametrize("rank_mode,scope", [(binding.RANK_POSITION, binding.SCOPE_HEAD),
                                             (binding.RANK_SCORE, binding.SCOPE_HEAD),
                                             (binding.RANK_SCORE, binding.SCOPE_LAYER)])
def test_static_scratch_selection_matches_workspace_selection_twice(rank_mode, scope):
    build.build()
    binding.lib()
    rng = np.random.default_rng(123)
    # two calls in a row with different shapes: the second sees the first one's leftovers in the scratch
    for lens, hkv, thr in [([3000, 17, 900], 4, 0.01), ([64, 5000], 2, 0.1)]:
        total = sum(lens)
        p = binding.Params(len(lens), hkv * 2, hkv, 128, window=16, sink=4, threshold=thr,
                           rank_mode=rank_mode, scope=scope)
        scores = torch.from_numpy((rng.random((hkv, total)) ** 6).astype(np.float32)).to(DEV)
        seq_len = torch.tensor(lens, dtype=torch.int32, device=DEV)
        want = _run(binding.refree_select_budget, p, scores, seq_len, total, True)
        got = _run(binding.refree_select_budget_static, p, scores, seq_len, total, False)
        rows = int(want[1][-1])
        assert 0 < rows < hkv * total
        assert torch.equal(got[0], want[0]) and torch.equal(got[1], want[1])
        assert torch.equal(got[2][:rows], want[2][:rows])


def test_static_scratch_limit_is_refused_before_any_launch():
    build.build()
    p = binding.Params(1024, 16, 16, 128, window=1)          # 16384 units need more than the built-in array
    assert 1024 * 16 * 24 > binding.STATIC_SCRATCH_BYTES
    rc = binding.refree_select_budget_static(p, torch.zeros(1, device=DEV), torch.zeros(1, dtype=torch.int32, device=DEV),
                                             1024, torch.zeros(1, dtype=torch.int32, device=DEV),
                                             torch.zeros(1, dtype=torch.int64, device=DEV), None, 0, check=False)
    assert rc == 8
    assert "built-in scratch" in binding.status_string(rc)
