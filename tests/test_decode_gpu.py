"""GPU parity of the decode-step attention over the compacted ragged cache
(the consumer of the pass) against the fp64 oracle, through the C ABI."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import refree_oracle as orc
from paper_2502_16886_b200 import binding, build, workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

# Products are exact (bf16 x bf16) or fp32, the softmax and all sums are fp32, the probabilities
# enter the second product as two bf16 terms (relative error 2^-17): the result is within a few
# 1e-5 of the row's sum of |p v|, which is at most max |v| ~ 5 for N(0, 1) rows.
ATOL, RTOL = 1e-4, 1e-4


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    binding.lib()


def run_decode(p, q_new, k_c, v_c, offsets, max_rows):
    ws = torch.empty(binding.refree_decode_workspace_size(p, max_rows) + 256, dtype=torch.uint8, device=DEV)
    out = torch.full((p.num_seqs, p.num_q_heads, p.head_dim), float("nan"), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    binding.refree_decode_attention(p, q_new.to(DEV), k_c.to(DEV), v_c.to(DEV), offsets.to(DEV), max_rows, out, ws,
                                    device_status=status)
    torch.cuda.synchronize()
    return out.cpu().numpy(), int(status.item())


def check_against_oracle(B, Hq, Hkv, d, dtype, lengths, seed, max_rows=None):
    tdt = torch.float32 if dtype == "fp32" else torch.bfloat16
    k_c, v_c, offsets = workloads.make_ragged_cache(seed, lengths, d, tdt)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed + 1)
    q_new = torch.randn((B, Hq, d), generator=gen, dtype=torch.float32).to(tdt)
    p = binding.Params(num_seqs=B, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=d,
                       dtype=binding.DTYPE_F32 if dtype == "fp32" else binding.DTYPE_BF16)
    got, status = run_decode(p, q_new, k_c, v_c, offsets, max(lengths) if max_rows is None else max_rows)
    op = orc.OracleParams(B, Hq, Hkv, d, dtype=0 if dtype == "fp32" else 1)
    want = orc.decode_attention(op, q_new, k_c, v_c, offsets.numpy())
    assert status == 0
    assert np.isfinite(got).all()
    np.testing.assert_allclose(got, want, rtol=RTOL, atol=ATOL)
    return got, want


@pytest.mark.parametrize("hq,hkv", [(8, 2), (7, 1), (32, 2), (3, 3)])
@pytest.mark.parametrize("d", [64, 128])
def test_bf16_ragged_segments_one_block_per_unit(hq, hkv, d):
    # empty, single-row, below / at / above one 16-row block, several warps' worth, a ragged tail
    B = 4
    base = [0, 1, 15, 16, 17, 129, 300, 1000, 33, 2, 128, 511]
    lengths = [base[i % len(base)] for i in range(B * hkv)]
    check_against_oracle(B, hq, hkv, d, "bf16", lengths, seed=11)


@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 128), (16, 1, 128), (12, 2, 64)])
def test_bf16_long_segments_split_over_blocks(hq, hkv, d):
    # few units: every unit is cut into many spans, merged by the second kernel
    lengths = [5000, 4097][:hkv] if hkv == 2 else [6001]
    check_against_oracle(1, hq, hkv, d, "bf16", lengths, seed=12)
    # a bound far above the real lengths: most blocks of the grid have no rows
    check_against_oracle(1, hq, hkv, d, "bf16", lengths, seed=13, max_rows=20000)
    # mixed: one unit empty, one inside a single span
    mixed = ([0, 3000] if hkv == 2 else [70])
    check_against_oracle(1, hq, hkv, d, "bf16", mixed, seed=14, max_rows=3000)


@pytest.mark.parametrize("dtype,d,hq,hkv", [("fp32", 64, 4, 2), ("fp32", 128, 6, 2), ("fp32", 64, 16, 1)])
def test_fp32_cache(dtype, d, hq, hkv):
    lengths = [0, 1, 40, 700, 129, 16][: 3 * hkv]
    check_against_oracle(3, hq, hkv, d, dtype, lengths, seed=15)
    check_against_oracle(1, hq, hkv, d, dtype, [2500, 1777][:hkv], seed=16)


def test_one_hot_and_uniform_attention():
    # a key aligned with the query and scaled up takes all the weight: out = its value row;
    # identical keys give uniform weights: out = the mean of the value rows
    d, n = 128, 600
    k_c, v_c, offsets = workloads.make_ragged_cache(21, [n, n], d, torch.bfloat16)
    q_new = torch.zeros((1, 2, d), dtype=torch.bfloat16)
    q_new[0, 0, 3] = 16.0
    k_c[:n] = 0
    k_c[417, 3] = 64.0                                # logit 1024 / sqrt(128) ~ 90 above the rest
    q_new[0, 1] = 1.0
    k_c[n:] = k_c[n]                                  # all keys of the second unit equal
    p = binding.Params(num_seqs=1, num_q_heads=2, num_kv_heads=2, head_dim=d, dtype=binding.DTYPE_BF16)
    got, status = run_decode(p, q_new, k_c, v_c, offsets, n)
    assert status == 0
    np.testing.assert_allclose(got[0, 0], v_c[417].float().numpy(), rtol=0, atol=1e-6)
    np.testing.assert_allclose(got[0, 1], v_c[n:].double().mean(0).numpy(), rtol=1e-4, atol=1e-5)


def test_segment_longer_than_the_stated_bound_is_flagged():
    k_c, v_c, offsets = workloads.make_ragged_cache(31, [400, 100], 128, torch.bfloat16)
    q_new = torch.ones((1, 2, 128), dtype=torch.bfloat16)
    p = binding.Params(num_seqs=1, num_q_heads=2, num_kv_heads=2, head_dim=128, dtype=binding.DTYPE_BF16)
    _, status = run_decode(p, q_new, k_c, v_c, offsets, 128)
    assert status & binding.DEV_CAPACITY


def test_argument_checks():
    p = binding.Params(num_seqs=1, num_q_heads=2, num_kv_heads=2, head_dim=128, dtype=binding.DTYPE_BF16)
    k_c, v_c, offsets = workloads.make_ragged_cache(41, [40, 10], 128, torch.bfloat16)
    q = torch.ones((1, 2, 128), dtype=torch.bfloat16, device=DEV)
    out = torch.zeros((1, 2, 128), dtype=torch.float32, device=DEV)
    ws = torch.empty(binding.refree_decode_workspace_size(p, 40) + 256, dtype=torch.uint8, device=DEV)
    kd, vd, od = k_c.to(DEV), v_c.to(DEV), offsets.to(DEV)
    assert binding.refree_decode_attention(p, q, kd, vd, od, 40, out, ws[:16], check=False) == binding.ERR_WORKSPACE
    assert binding.refree_decode_attention(p, q, None, vd, od, 40, out, ws, check=False) == binding.ERR_INVALID_ARG
    bad = dataclasses.replace(p, head_dim=96)
    assert binding.refree_decode_attention(bad, q, kd, vd, od, 40, out, ws, check=False) == binding.ERR_UNSUPPORTED
    many = dataclasses.replace(p, num_q_heads=34)      # 17 query heads per KV head
    assert binding.refree_decode_attention(many, q, kd, vd, od, 40, out, ws, check=False) == binding.ERR_UNSUPPORTED


@pytest.mark.parametrize("rank_mode", [binding.RANK_POSITION, binding.RANK_SCORE])
def test_decode_consumes_the_output_of_the_pass(rank_mode):
    # compress a layer, then attend over what came out; the oracle does the same on its own output
    cfg = dataclasses.replace(workloads.CONFIGS[0], dtype="bf16", head_dim=128, num_q_heads=8, num_kv_heads=2, window=8)
    lay = workloads.make_layer(cfg, 0, seq_lens=[900, 37, 260])
    p = binding.params_for(cfg, lay, rank_mode=rank_mode, threshold=0.05)
    res = binding.compress_layer(p, lay.q_win.to(DEV), lay.k.to(DEV), lay.v.to(DEV), lay.seq_start.to(DEV),
                                 lay.seq_len.to(DEV), lay.total_tokens)
    q_new = workloads.make_decode_query(cfg, 0, lay.q_win)
    rows = int(res.offsets[-1].item())
    got, status = run_decode(p, q_new, res.k_out[:max(rows, 1)], res.v_out[:max(rows, 1)], res.offsets,
                             int(lay.seq_len.max().item()))
    assert status == 0
    op = orc.OracleParams(p.num_seqs, p.num_q_heads, p.num_kv_heads, p.head_dim, dtype=1)
    want = orc.decode_attention(op, q_new, res.k_out[:max(rows, 1)].cpu(), res.v_out[:max(rows, 1)].cpu(),
                                res.offsets.cpu().numpy())
    np.testing.assert_allclose(got, want, rtol=RTOL, atol=ATOL)
