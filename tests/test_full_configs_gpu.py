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
    print(f"{name} layer {layer} rank_mode {rank_mode}: {ties} of {units} units under the near-tie rule, "
          f"worst score error {worst:.2e} relative")
    # observed on every config and both rankings: no unit needs the near-tie rule (budgets and kept sets equal the
    # oracle's outright), and the scores agree to 1e-6; a regression in either shows here, not behind a loose bound
    assert ties == 0, f"{ties} of {units} units needed the near-tie rule"
    assert worst < 1e-5
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


@pytest.mark.parametrize("name,n_layers", [("mistral7b_32k", 4), ("qwen25_7b_ragged8", 3)])
def test_one_call_run_of_layers_at_full_size(name, n_layers):
    """The step the benchmark times: refree_compress_layers over consecutive full-size layers (both
    workspace halves reused).  Budgets and every compacted row against the oracle (every layer's budgets equal
    the oracle's on these workloads), and against the per-layer call, which must agree with the one-call run
    bit for bit in any case."""
    from oracle import refree_oracle as orc
    cfg = workloads.get_config(name)
    dev = "cuda:0"
    lays = [workloads.make_layer(cfg, l) for l in range(n_layers)]
    p = binding.params_for(cfg, lays[0])
    total = lays[0].total_tokens
    cap = p.num_kv_heads * total
    units = p.num_seqs * p.num_kv_heads
    q = [l.q_win.to(dev) for l in lays]
    k = [l.k.to(dev) for l in lays]
    v = [l.v.to(dev) for l in lays]
    k_out = [torch.zeros(cap, p.head_dim, dtype=lays[0].k.dtype, device=dev) for _ in lays]
    v_out = [torch.zeros(cap, p.head_dim, dtype=lays[0].k.dtype, device=dev) for _ in lays]
    lengths = [torch.zeros(units, dtype=torch.int32, device=dev) for _ in lays]
    offsets = [torch.zeros(units + 1, dtype=torch.int64, device=dev) for _ in lays]
    ss, sl = lays[0].seq_start.to(dev), lays[0].seq_len.to(dev)
    ws = torch.empty(binding.refree_layers_workspace_size(p, total), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    binding.refree_compress_layers(p, binding.LayerPointers(q, k, v, k_out, v_out, lengths, offsets), ss, sl, total, cap,
                                   ws, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    exact = 0
    for l, lay in enumerate(lays):
        one = binding.compress_layer(p, q[l], k[l], v[l], ss, sl, total, want_scores=False, want_kept_idx=False)
        torch.cuda.synchronize()
        rows = int(offsets[l][-1])
        assert torch.equal(lengths[l], one.lengths.reshape(-1)) and torch.equal(offsets[l], one.offsets)
        assert torch.equal(parity.bits(k_out[l][:rows]), parity.bits(one.k_out[:rows]))
        assert torch.equal(parity.bits(v_out[l][:rows]), parity.bits(one.v_out[:rows]))
        ref = orc.compress_layer(parity.oracle_params(p), lay.q_win, lay.k, lay.v, lay.seq_start, lay.seq_len)
        if np.array_equal(lengths[l].cpu().numpy(), ref.sel.lengths.reshape(-1)):
            exact += 1
            assert rows == int(ref.sel.offsets[-1])
            assert torch.equal(parity.bits(k_out[l][:rows].cpu()), parity.bits(ref.k_out))
            assert torch.equal(parity.bits(v_out[l][:rows].cpu()), parity.bits(ref.v_out))
        del one
    assert exact == n_layers, f"only {exact} of {n_layers} layers had the oracle's budgets exactly"
    torch.cuda.empty_cache()
