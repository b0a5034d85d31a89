"""Full-size parity: one layer of every benchmark config, in the launch
configuration the benchmark times (fused pass, head-major cache), compared with
the oracle in full - scores element by element, budgets, kept sets, and the
compacted K/V bit for bit."""
import numpy as np
import pytest
import torch

from paper_2502_16886_b200 import binding, build, workloads
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


@pytest.mark.parametrize("rank_mode", [binding.RANK_POSITION, binding.RANK_SCORE])
@pytest.mark.parametrize("name,layer", [("tiny", 0), ("llama3_8b_8k", 0), ("mistral7b_32k", 0), ("mistral7b_32k", 1),
                                        ("qwen25_7b_ragged8", 0), ("llama3_70b_20k", 0)])
def test_full_size_layer_matches_oracle(name, layer, rank_mode):
    cfg = workloads.get_config(name)
    lay = workloads.make_layer(cfg, layer)
    res, ref, worst, ties = parity.run_fused_and_check(cfg, lay, rank_mode=rank_mode)
    units = res.lengths.numel()
    assert ties <= max(1, units // 4), f"{ties} of {units} units needed the near-tie rule"
    rho = float(res.lengths.sum()) / (cfg.num_kv_heads * lay.total_tokens)
    assert 0.0 < rho <= 1.0
    torch.cuda.empty_cache()


def test_layer_scope_and_frozen_layer_at_full_size():
    cfg = workloads.get_config("llama3_8b_8k")
    lay = workloads.make_layer(cfg, 2)
    res, ref, _, _ = parity.run_fused_and_check(cfg, lay, scope=binding.SCOPE_LAYER)
    assert len(set(res.lengths.cpu().reshape(-1).tolist())) == 1      # one budget for the layer
    res, _, _, _ = parity.run_fused_and_check(cfg, lay, force_full=1, want_scores=False)
    assert (res.lengths == 8192).all()


@pytest.mark.parametrize("name", ["llama3_8b_8k", "mistral7b_32k", "qwen25_7b_ragged8", "llama3_70b_20k"])
def test_decode_attention_over_the_compacted_layer_at_full_size(name):
    # the consumer of the pass at benchmark size: every output element against the fp64 oracle
    from oracle import refree_oracle as orc
    cfg = workloads.get_config(name)
    lay = workloads.make_layer(cfg, 0)
    dev = "cuda:0"
    p = binding.params_for(cfg, lay)
    res = binding.compress_layer(p, lay.q_win.to(dev), lay.k.to(dev), lay.v.to(dev), lay.seq_start.to(dev),
                                 lay.seq_len.to(dev), lay.total_tokens, want_scores=False, want_kept_idx=False)
    q_new = workloads.make_decode_query(cfg, 0, lay.q_win)
    max_rows = int(lay.seq_len.max().item())
    ws = torch.empty(binding.refree_decode_workspace_size(p, max_rows), dtype=torch.uint8, device=dev)
    out = torch.empty((p.num_seqs, p.num_q_heads, p.head_dim), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    binding.refree_decode_attention(p, q_new.to(dev), res.k_out, res.v_out, res.offsets, max_rows, out, ws,
                                    device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rows = int(res.offsets[-1].item())
    op = orc.OracleParams(p.num_seqs, p.num_q_heads, p.num_kv_heads, p.head_dim, dtype=1)
    want = orc.decode_attention(op, q_new, res.k_out[:rows].cpu(), res.v_out[:rows].cpu(), res.offsets.cpu().numpy())
    np.testing.assert_allclose(out.cpu().numpy(), want, rtol=1e-4, atol=1e-4)
    torch.cuda.empty_cache()
