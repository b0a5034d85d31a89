"""Pins for the CPU oracle: everything here checks ``oracle/`` against something
that is not the oracle — the paper's definitions evaluated by brute force with
numpy on tiny inputs, closed forms, invariants, library routines."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import refree_oracle as orc

T32 = float(np.float32(0.01))


def _params(B, Hq, Hkv, d, w, n_total, **kw):
    dtype = kw.pop("dtype", 0)
    p = orc.OracleParams(B, Hq, Hkv, d, window=w, dtype=dtype, **kw)
    p.k_strides = (0, d, n_total * d)      # head-major [Hkv, N, d]
    p.v_strides = (0, d, n_total * d)
    return p


# ---------------------------------------------------------------- scoring ----
def _brute_scores(q_full, k, G, w):
    """Literal reading of Section 3.2: A = causal softmax(Q K^T / sqrt(d)), n x n,
    per query head; Eq. 2 reduces its last w rows, dividing each column by its
    count of non-zero entries; a KV head takes the mean over its query heads."""
    Hq, n, d = q_full.shape
    Hkv = Hq // G
    out = np.zeros((Hkv, n))
    for h in range(Hq):
        logits = q_full[h] @ k[h // G].T / math.sqrt(d)
        logits = np.where(np.tril(np.ones((n, n), dtype=bool)), logits, -np.inf)
        A = np.exp(logits - logits.max(axis=1, keepdims=True))
        A = A / A.sum(axis=1, keepdims=True)
        last = A[max(0, n - w):]
        nz = (last != 0).sum(axis=0)
        out[h // G] += last.sum(axis=0) / nz
    return out / G


@pytest.mark.parametrize("n,w,G,Hkv,d", [(48, 8, 2, 2, 16), (33, 1, 4, 1, 8), (64, 64, 1, 2, 8),
                                         (5, 16, 2, 1, 8), (1, 4, 2, 2, 8), (40, 7, 3, 2, 24)])
def test_score_matches_full_attention_matrix(n, w, G, Hkv, d):
    rng = np.random.default_rng(n * 1000 + w)
    Hq = G * Hkv
    q_full = rng.standard_normal((Hq, n, d)).astype(np.float32)
    k = (1.5 * rng.standard_normal((Hkv, n, d))).astype(np.float32)
    want = _brute_scores(q_full.astype(np.float64), k.astype(np.float64), G, w)
    # window block: row r of q_win is the query at position n - w + r
    q_win = rng.standard_normal((1, Hq, w, d)).astype(np.float32) * 50.0   # junk where pos < 0
    w_eff = min(w, n)
    q_win[0, :, w - w_eff:, :] = q_full[:, n - w_eff:, :]
    p = _params(1, Hq, Hkv, d, w, n)
    got = orc.score(p, torch.from_numpy(q_win), torch.from_numpy(k), [0], [n])
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-300)


def test_score_single_row_is_textbook_softmax():
    from scipy.special import softmax
    rng = np.random.default_rng(7)
    n, d = 100, 32
    q = rng.standard_normal((1, 1, 1, d)).astype(np.float32)
    k = rng.standard_normal((1, n, d)).astype(np.float32)
    p = _params(1, 1, 1, d, 1, n)
    got = orc.score(p, torch.from_numpy(q), torch.from_numpy(k), [0], [n])[0]
    want = softmax(k[0].astype(np.float64) @ q[0, 0, 0].astype(np.float64) / math.sqrt(d))
    np.testing.assert_allclose(got, want, rtol=1e-12)
    assert abs(got.sum() - 1.0) < 1e-12


def test_score_column_mass_identity_ragged_batch_bf16_and_strides():
    """Each window row is a probability vector, so sum_i a'[i]*cnt(i) = w_eff for
    every KV head; also exercises bf16 storage, a ragged batch and both layouts."""
    rng = np.random.default_rng(3)
    lens = [70, 9, 33]
    B, Hq, Hkv, d, w = 3, 4, 2, 16, 12
    N = sum(lens)
    starts = np.concatenate([[0], np.cumsum(lens)[:-1]]).astype(np.int32)
    k_hm = torch.from_numpy(rng.standard_normal((Hkv, N, d)).astype(np.float32)).to(torch.bfloat16)
    q = torch.from_numpy(rng.standard_normal((B, Hq, w, d)).astype(np.float32)).to(torch.bfloat16)
    p = _params(B, Hq, Hkv, d, w, N, dtype=1)
    a = orc.score(p, q, k_hm, starts, lens)
    off = 0
    for n in lens:
        w_eff = min(w, n)
        cnt = np.minimum(w_eff, n - np.arange(n))
        for g in range(Hkv):
            assert abs((a[g, off:off + n] * cnt).sum() - w_eff) < 1e-10
        off += n
    # token-major layout of the same cache gives the same scores
    k_tm = k_hm.permute(1, 0, 2).contiguous()
    p2 = _params(B, Hq, Hkv, d, w, N, dtype=1)
    p2.k_strides = (0, Hkv * d, d)
    a2 = orc.score(p2, q, k_tm, starts, lens)
    np.testing.assert_array_equal(a, a2)
    # bf16 bits are widened exactly: fp32 copies of the same values score the same
    p3 = _params(B, Hq, Hkv, d, w, N, dtype=0)
    a3 = orc.score(p3, q.float(), k_hm.float(), starts, lens)
    np.testing.assert_array_equal(a, a3)
    # a sequence scored alone equals its slice of the batch (units are independent)
    p4 = _params(1, Hq, Hkv, d, w, N, dtype=1)
    a4 = orc.score(p4, q[1:2], k_hm, [int(starts[1])], [lens[1]])
    np.testing.assert_array_equal(a4, a[:, lens[0]:lens[0] + lens[1]])


def test_score_uniform_when_queries_are_zero():
    n, d, w = 40, 8, 4
    k = torch.randn(1, n, d)
    q = torch.zeros(1, 2, w, d)
    p = _params(1, 2, 1, d, w, n)
    a = orc.score(p, q, k, [0], [n])[0]
    # row at position r is uniform over r+1 keys; Eq. 2 averages the visible rows
    rows = [np.concatenate([np.full(r + 1, 1.0 / (r + 1)), np.zeros(n - r - 1)]) for r in range(n - w, n)]
    want = np.sum(rows, axis=0) / np.minimum(w, n - np.arange(n))
    np.testing.assert_allclose(a, want, rtol=1e-13)


# -------------------------------------------------------------- selection ----
def _paper_position_order(n, m):
    """X_hat = {x_1..x_m, x_n, x_{n-1}, .., x_{m+1}} (Section 3.2), 0-based."""
    m = min(m, n)
    one_based = list(range(1, m + 1)) + list(range(n, m, -1))
    return np.array(one_based) - 1


def _score_order(sq, n, m, w_eff):
    m = min(m, n)
    if m + w_eff >= n:
        return np.arange(n)
    rest = np.arange(m, n - w_eff)
    order = rest[np.argsort(-sq[rest], kind="stable")]
    return np.concatenate([np.arange(m), np.arange(n - w_eff, n), order])


def _brute_stop(sq_ranked, T):
    """Eq. 1 by its definition: for every j mask out ranked positions > j and take
    the norm of what is left; leftmost j with 1 - |A_j|/|A| < T, else n."""
    n = len(sq_ranked)
    a = np.sqrt(sq_ranked)
    full = np.linalg.norm(a)
    for j in range(1, n + 1):
        masked = np.where(np.arange(n) < j, a, 0.0)
        if full > 0 and 1.0 - np.linalg.norm(masked) / full < T:
            return j
    return n


@pytest.mark.parametrize("rank_mode", [0, 1])
@pytest.mark.parametrize("scope", [0, 1])
@pytest.mark.parametrize("T", [0.01, 0.1, 0.35])
def test_select_matches_masked_norm_definition(rank_mode, scope, T):
    rng = np.random.default_rng(11 + rank_mode * 7 + scope)
    lens = [37, 12, 3, 50]
    B, Hkv, m, w = len(lens), 3, 4, 5
    N = sum(lens)
    sc = (rng.random((Hkv, N)) ** 4).astype(np.float32)       # skewed, tie-free
    p = orc.OracleParams(B, Hkv, Hkv, 8, window=w, sink=m, threshold=T, rank_mode=rank_mode,
                         scope=scope, keep_window=0)
    sel = orc.select(p, sc, lens)
    Tf = float(np.float32(T))
    off = 0
    for s, n in enumerate(lens):
        w_eff = min(w, n)
        for g in range(Hkv):
            if scope == 0:
                sq = sc[g, off:off + n].astype(np.float64) ** 2
            else:
                sq = (sc[:, off:off + n].astype(np.float64) ** 2).sum(axis=0)
            order = _paper_position_order(n, m) if rank_mode == 0 else _score_order(sq, n, m, w_eff)
            np.testing.assert_array_equal(sel.pi[g, off:off + n], order)
            j = _brute_stop(sq[order], Tf)
            assert sel.jstar[s, g] == j
            assert sel.lengths[s, g] == max(j, 1)
            u = s * Hkv + g
            kept = sel.kept_idx[sel.offsets[u]:sel.offsets[u + 1]]
            np.testing.assert_array_equal(kept, np.sort(order[:max(j, 1)]))
            # the criterion curve sqrt(C_j / C_n) of Eq. 3 and the distance of the decision from a tie: the
            # parity rules excuse a budget mismatch only through these two, so they are pinned like the rest
            curve = np.sqrt(np.cumsum(sq[order]) / sq.sum())
            np.testing.assert_allclose(sel.ratio[g, off:off + n], curve, rtol=1e-13, atol=0)
            crossed = (1.0 - curve < Tf).any()
            if crossed:
                near = [abs(curve[j - 1] - (1.0 - Tf))] + ([abs(curve[j - 2] - (1.0 - Tf))] if j > 1 else [])
                want_gap = min(near)
            else:
                want_gap = abs(1.0 - (1.0 - Tf))
            np.testing.assert_allclose(sel.gap[s, g], want_gap, rtol=1e-9, atol=1e-15)
        off += n
    np.testing.assert_array_equal(sel.offsets, np.concatenate([[0], np.cumsum(sel.lengths.reshape(-1))]))


@pytest.mark.parametrize("n", [512, 8192, 32768, 20480])
def test_stop_index_uniform_scores_closed_form(n):
    """All squares equal: C_j/C_n = j/n, so j* = floor((1-T)^2 n) + 1."""
    p = orc.OracleParams(1, 1, 1, 8, window=1, sink=4, threshold=0.01, keep_window=0)
    sel = orc.select(p, np.full((1, n), 0.25, dtype=np.float32), [n])
    assert sel.jstar[0, 0] == math.floor((1.0 - T32) ** 2 * n) + 1
    assert {512: 502, 8192: 8029, 32768: 32116, 20480: 20073}[n] == sel.jstar[0, 0]


@pytest.mark.parametrize("rank_p", [1, 3, 4, 5, 17, 64])
def test_stop_index_one_hot_is_its_rank(rank_p):
    n, m = 64, 4
    order = _paper_position_order(n, m)
    sc = np.zeros((1, n), dtype=np.float32)
    sc[0, order[rank_p - 1]] = 0.7
    p = orc.OracleParams(1, 1, 1, 8, window=1, sink=m, threshold=0.01, keep_window=0)
    assert orc.select(p, sc, [n]).jstar[0, 0] == rank_p


@pytest.mark.parametrize("c,T", [(0.9, 0.01), (0.97, 0.05), (0.5, 0.001)])
def test_stop_index_geometric_closed_form(c, T):
    """a'[pi_j] = c^j: C_j/C_n = (1-c^(2j))/(1-c^(2n)); j* = floor(x)+1 with
    x = ln(1-(1-T)^2 (1-c^(2n))) / (2 ln c)."""
    n, m = 200, 4
    order = _paper_position_order(n, m)
    sc = np.zeros((1, n), dtype=np.float32)
    sc[0, order] = (c ** np.arange(1, n + 1)).astype(np.float32)
    Tf = float(np.float32(T))
    x = math.log(1.0 - (1.0 - Tf) ** 2 * (1.0 - c ** (2 * n))) / (2.0 * math.log(c))
    assert abs(x - round(x)) > 1e-3          # the closed form is not at a tie
    p = orc.OracleParams(1, 1, 1, 8, window=1, sink=m, threshold=T, keep_window=0)
    assert orc.select(p, sc, [n]).jstar[0, 0] == math.floor(x) + 1


def test_budget_monotone_in_threshold_and_scale_invariant():
    rng = np.random.default_rng(5)
    n = 300
    sc = (rng.random((2, n)) ** 6).astype(np.float32)
    prev = None
    for T in [0.0, 1e-4, 1e-3, 0.01, 0.05, 0.2, 0.6, 0.99]:
        for mode in (0, 1):
            p = orc.OracleParams(1, 2, 2, 8, window=8, sink=4, threshold=T, rank_mode=mode, keep_window=0)
            b = orc.select(p, sc, [n]).lengths
            b2 = orc.select(p, (sc * np.float32(0.125)), [n]).lengths    # exact power-of-two scaling
            np.testing.assert_array_equal(b, b2)
            if mode == 0:
                if prev is not None:
                    assert (b <= prev).all()
                prev = b
    p0 = orc.OracleParams(1, 2, 2, 8, window=8, sink=4, threshold=0.0, keep_window=0)
    assert (orc.select(p0, sc, [n]).lengths == n).all()          # no j satisfies Eq. 1: keep all
    pz = orc.OracleParams(1, 2, 2, 8, window=8, sink=4, threshold=0.01, keep_window=0)
    assert (orc.select(pz, np.zeros((2, n), dtype=np.float32), [n]).lengths == n).all()   # C_n = 0


@pytest.mark.parametrize("rank_mode", [0, 1])
def test_window_floor_force_full_and_kept_set_shape(rank_mode):
    rng = np.random.default_rng(9)
    lens = [90, 6, 200]
    Hkv, m, w = 2, 4, 16
    N = sum(lens)
    sc = (rng.random((Hkv, N)) ** 8).astype(np.float32)
    sc[:, 0] = 1000.0        # a dominant sink: Eq. 1 alone would stop at j = 1
    sc[:, lens[0]] = 1000.0
    sc[:, lens[0] + lens[1]] = 1000.0
    base = dict(window=w, sink=m, threshold=0.01, rank_mode=rank_mode)
    lit = orc.select(orc.OracleParams(3, Hkv, Hkv, 8, keep_window=0, **base), sc, lens)
    assert (lit.lengths == 1).all()
    kw = orc.select(orc.OracleParams(3, Hkv, Hkv, 8, keep_window=1, **base), sc, lens)
    off = 0
    for s, n in enumerate(lens):
        w_eff = min(w, n)
        for g in range(Hkv):
            u = s * Hkv + g
            kept = kw.kept_idx[kw.offsets[u]:kw.offsets[u + 1]]
            assert kw.lengths[s, g] == min(n, m + w_eff)
            assert set(range(n - w_eff, n)) <= set(kept.tolist())
            assert set(range(min(m, n))) <= set(kept.tolist())
            assert (np.diff(kept) > 0).all()
        off += n
    ff = orc.select(orc.OracleParams(3, Hkv, Hkv, 8, force_full=1, **base), sc, lens)
    for s, n in enumerate(lens):
        for g in range(Hkv):
            u = s * Hkv + g
            np.testing.assert_array_equal(ff.kept_idx[ff.offsets[u]:ff.offsets[u + 1]], np.arange(n))


def test_position_mode_kept_set_is_prefix_plus_suffix():
    rng = np.random.default_rng(21)
    n, m = 500, 4
    sc = rng.random((1, n)).astype(np.float32)
    p = orc.OracleParams(1, 1, 1, 8, window=8, sink=m, threshold=0.1)
    sel = orc.select(p, sc, [n])
    b = int(sel.lengths[0, 0])
    assert m < b < n
    np.testing.assert_array_equal(sel.kept_idx, np.concatenate([np.arange(m), np.arange(n - (b - m), n)]))


def test_layer_scope_gives_one_integer_budget_per_layer_like_the_printed_ones():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_case_study_budgets.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    for _, n, pct, cnt in rows:
        assert round(100.0 * int(cnt) / int(n), 2) == float(pct)
    rng = np.random.default_rng(2)
    n, Hkv = 96, 8
    sc = (rng.random((Hkv, n)) ** 3).astype(np.float32)
    p = orc.OracleParams(1, Hkv, Hkv, 8, window=1, sink=4, threshold=0.01, scope=1)
    b = orc.select(p, sc, [n]).lengths
    assert (b == b[0, 0]).all()


# -------------------------------------------------------------- compaction ----
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("layout", ["head_major", "token_major"])
def test_compact_rows_are_bit_identical(dtype, layout):
    rng = np.random.default_rng(4)
    lens = [40, 17]
    B, Hkv, d = 2, 3, 16
    N = sum(lens)
    starts = [0, 40]
    k = torch.from_numpy(rng.standard_normal((Hkv, N, d)).astype(np.float32)).to(dtype)
    v = torch.from_numpy(rng.standard_normal((Hkv, N, d)).astype(np.float32)).to(dtype)
    sc = (rng.random((Hkv, N)) ** 5).astype(np.float32)
    p = orc.OracleParams(B, Hkv, Hkv, d, window=4, sink=2, threshold=0.05, rank_mode=1,
                         dtype=0 if dtype == torch.float32 else 1)
    if layout == "head_major":
        p.k_strides = p.v_strides = (0, d, N * d)
        kk, vv = k, v
    else:
        p.k_strides = p.v_strides = (0, Hkv * d, d)
        kk, vv = k.permute(1, 0, 2).contiguous(), v.permute(1, 0, 2).contiguous()
    sel = orc.select(p, sc, lens)
    k_out, v_out = orc.compact(p, kk, vv, starts, lens, sel)
    as_bits = (lambda t: t.view(torch.int32)) if dtype == torch.float32 else (lambda t: t.view(torch.int16))
    for s in range(B):
        for g in range(Hkv):
            u = s * Hkv + g
            idx = torch.from_numpy(sel.kept_idx[sel.offsets[u]:sel.offsets[u + 1]].astype(np.int64)) + starts[s]
            assert torch.equal(as_bits(k_out[sel.offsets[u]:sel.offsets[u + 1]]), as_bits(k[g, idx]))
            assert torch.equal(as_bits(v_out[sel.offsets[u]:sel.offsets[u + 1]]), as_bits(v[g, idx]))


def test_compress_layer_end_to_end_on_tiny_workload():
    from paper_2502_16886_b200 import workloads
    cfg = workloads.CONFIGS[0]
    lay = workloads.make_layer(cfg, 0)
    ss, st, sh = lay.strides()
    for mode in (0, 1):
        p = orc.OracleParams(1, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, window=cfg.window,
                             sink=cfg.sink, rank_mode=mode, dtype=0, k_strides=(ss, st, sh), v_strides=(ss, st, sh))
        res = orc.compress_layer(p, lay.q_win, lay.k, lay.v, lay.seq_start, lay.seq_len)
        n = cfg.seq_lens[0]
        assert res.scores.shape == (cfg.num_kv_heads, n)
        # heavy keys are the heaviest non-window positions of their head
        for g in range(cfg.num_kv_heads):
            body = res.scores[g, cfg.sink:n - cfg.window]
            top = set((np.argsort(-body)[:len(lay.heavy_idx[0][g])] + cfg.sink).tolist())
            assert top == set(lay.heavy_idx[0][g].tolist())
        assert (res.sel.lengths >= cfg.sink + cfg.window).all() and (res.sel.lengths <= n).all()
        if mode == 1:      # ranking by score keeps the heaviest keys first
            for g in range(cfg.num_kv_heads):
                kept = set(res.sel.kept_idx[res.sel.offsets[g]:res.sel.offsets[g + 1]].tolist())
                extra = int(res.sel.lengths[0, g]) - cfg.sink - cfg.window
                body = res.scores32[g, cfg.sink:n - cfg.window]
                want = set((np.argsort(-body, kind="stable")[:extra] + cfg.sink).tolist())
                assert kept == want | set(range(cfg.sink)) | set(range(n - cfg.window, n))


# --------------------------------------------------------- decode consumer ----
def test_decode_attention_matches_numpy_softmax_attention():
    from scipy.special import softmax
    rng = np.random.default_rng(8)
    B, Hq, Hkv, d = 2, 4, 2, 16
    lengths = np.array([5, 9, 1, 7])
    offsets = np.concatenate([[0], np.cumsum(lengths)])
    k_c = rng.standard_normal((offsets[-1], d)).astype(np.float32)
    v_c = rng.standard_normal((offsets[-1], d)).astype(np.float32)
    q = rng.standard_normal((B, Hq, d)).astype(np.float32)
    p = orc.OracleParams(B, Hq, Hkv, d, dtype=0)
    got = orc.decode_attention(p, torch.from_numpy(q), torch.from_numpy(k_c), torch.from_numpy(v_c), offsets)
    for s in range(B):
        for h in range(Hq):
            u = s * Hkv + h // (Hq // Hkv)
            ks, vs = k_c[offsets[u]:offsets[u + 1]].astype(np.float64), v_c[offsets[u]:offsets[u + 1]].astype(np.float64)
            pr = softmax(ks @ q[s, h].astype(np.float64) / math.sqrt(d))
            np.testing.assert_allclose(got[s, h], pr @ vs, rtol=1e-12, atol=1e-14)
