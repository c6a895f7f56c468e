"""Pins for the CPU oracle: brute force, closed forms and invariants fixed by the paper's equations.

Each pin is independent of the oracle's own formula: pure-Python loops with ``math.exp``, hand-derived
closed forms (tests/golden/softmax_closed_forms.txt), a library fp64 attention as a second opinion,
and the invariants of Eq. 1, 2, 8, 9, 10 and 11.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import avsa_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "softmax_closed_forms.txt")


def _golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, v = line.split()
            out[k] = float(v)
    return out


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


# ------------------------------------------------------------------------------- Eq. 1 / Eq. 2
def _brute_cross(q, k, v, scale):
    """Pure-Python triple loop of Eq. 1 for one head: q [Nq][d], k,v [Nk][d]."""
    nq, nk, d = len(q), len(k), len(q[0])
    O = [[0.0] * d for _ in range(nq)]
    A = [[0.0] * nk for _ in range(nq)]
    lse = [0.0] * nq
    for j in range(nq):
        logits = [sum(q[j][t] * k[i][t] for t in range(d)) * scale for i in range(nk)]
        z = sum(math.exp(x) for x in logits)          # no max shift: small inputs
        lse[j] = math.log(z)
        for i in range(nk):
            A[j][i] = math.exp(logits[i]) / z
            for t in range(d):
                O[j][t] += A[j][i] * v[i][t]
    return O, lse, A


def test_cross_attention_brute_force():
    B, H, Nq, Nk, d = 2, 2, 3, 7, 5
    q, k, v = _rand((B, H, Nq, d), 1), _rand((B, H, Nk, d), 2), _rand((B, H, Nk, d), 3)
    O, lse, A = orc.cross_attention(q, k, v)
    for b in range(B):
        for h in range(H):
            Ob, lb, Ab = _brute_cross(q[b, h].tolist(), k[b, h].tolist(), v[b, h].tolist(), 1 / math.sqrt(d))
            np.testing.assert_allclose(O[b, h], Ob, rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(lse[b, h], lb, rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(A[b, h], Ab, rtol=1e-12, atol=1e-14)


def test_cross_attention_golden_closed_form():
    g = _golden()
    q = np.array([[[[1.0], [1.0]]]])
    k = np.array([[[[0.0], [math.log(3.0)], [math.log(4.0)]]]])
    v = np.array([[[[8.0], [16.0], [24.0]]]])
    O, lse, A = orc.cross_attention(q, k, v, scale=1.0)
    np.testing.assert_allclose(A[0, 0, 0], [g["dense_p0"], g["dense_p1"], g["dense_p2"]], rtol=1e-14)
    np.testing.assert_allclose(O[0, 0, :, 0], [g["dense_out"]] * 2, rtol=1e-14)
    np.testing.assert_allclose(lse[0, 0], [g["dense_lse"]] * 2, rtol=1e-14)
    s = orc.column_scores(A)
    np.testing.assert_allclose(s[0], [g["colsum0"], g["colsum1"], g["colsum2"]], rtol=1e-14)


def test_cross_attention_rows_sum_to_one_and_column_mass():
    B, H, Nq, Nk, d = 2, 3, 9, 50, 16
    q, k, v = _rand((B, H, Nq, d), 4) * 3, _rand((B, H, Nk, d), 5), _rand((B, H, Nk, d), 6)
    _, _, A = orc.cross_attention(q, k, v)
    np.testing.assert_allclose(A.sum(-1), 1.0, atol=1e-12)
    s = orc.column_scores(A)
    np.testing.assert_allclose(s.sum(-1), H * Nq, rtol=1e-12)                       # Eq. 2 mass
    s1 = orc.column_scores(A, gamma=1.0 / (H * Nq))
    np.testing.assert_allclose(s1.sum(-1), 1.0, rtol=1e-12)                         # L1 Norm
    prev = _rand((B, Nk), 7)
    s2 = orc.column_scores(A, s_prev=prev, beta=0.25, gamma=0.75)
    np.testing.assert_allclose(s2, 0.25 * prev + 0.75 * s, rtol=1e-13)


def test_cross_attention_identical_keys_closed_form():
    B, H, Nq, Nk, d = 1, 2, 4, 11, 8
    q = _rand((B, H, Nq, d), 8)
    k = np.broadcast_to(_rand((B, H, 1, d), 9), (B, H, Nk, d)).copy()
    v = _rand((B, H, Nk, d), 10)
    O, lse, A = orc.cross_attention(q, k, v)
    np.testing.assert_allclose(A, 1.0 / Nk, rtol=1e-12)
    np.testing.assert_allclose(O, np.broadcast_to(v.mean(2, keepdims=True), O.shape), rtol=1e-12, atol=1e-13)
    logit = (q * k[:, :, :1]).sum(-1) / math.sqrt(d)
    np.testing.assert_allclose(lse, logit + math.log(Nk), rtol=1e-12)
    np.testing.assert_allclose(orc.column_scores(A), H * Nq / Nk, rtol=1e-12)


def test_cross_attention_dominant_key_is_one_hot():
    d = 4
    q = np.ones((1, 1, 2, d))
    k = np.zeros((1, 1, 5, d)); k[0, 0, 3] = 100.0
    v = _rand((1, 1, 5, d), 11)
    O, _, A = orc.cross_attention(q, k, v)
    np.testing.assert_allclose(A[0, 0, :, 3], 1.0, atol=1e-12)
    np.testing.assert_allclose(O[0, 0], np.stack([v[0, 0, 3]] * 2), atol=1e-10)


def test_cross_attention_matches_library_fp64():
    B, H, Nq, Nk, d = 2, 2, 6, 33, 16
    q, k, v = _rand((B, H, Nq, d), 12), _rand((B, H, Nk, d), 13), _rand((B, H, Nk, d), 14)
    O, _, _ = orc.cross_attention(q, k, v)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v)).numpy()
    np.testing.assert_allclose(O, ref, rtol=1e-10, atol=1e-12)


# ------------------------------------------------------------------------------- Eq. 3 / Eq. 8
def _brute_topk(x, k):
    def key(i):
        val = x[i]
        if val != val:
            val = -math.inf
        return (-val, i)
    return sorted(range(len(x)), key=key)[:k]


def test_topk_matches_sorted_brute_force_with_ties():
    rng = np.random.default_rng(15)
    for trial in range(50):
        n = int(rng.integers(1, 40))
        x = rng.integers(-3, 4, size=n).astype(np.float64)          # many ties
        k = int(rng.integers(0, n + 1))
        assert orc.topk_indices(x, k).tolist() == _brute_topk(x.tolist(), k)


def test_topk_special_values():
    assert orc.topk_indices(np.ones(9), 4).tolist() == [0, 1, 2, 3]            # all equal
    assert orc.topk_indices(np.arange(5.0), 5).tolist() == [4, 3, 2, 1, 0]     # k = n
    assert orc.topk_indices(np.arange(5.0), 0).tolist() == []                  # k = 0
    x = np.array([np.nan, -0.0, 0.0, -np.inf, 1.0, np.nan])
    assert orc.topk_indices(x, 6).tolist() == [4, 1, 2, 0, 3, 5]               # -0 == +0, NaN == -inf
    x = np.array([2.0, 5.0, 2.0, 2.0, 7.0])                                    # threshold duplicated
    assert orc.topk_indices(x, 3).tolist() == [4, 1, 0]
    assert orc.topk_indices(x, 4).tolist() == [4, 1, 0, 2]


def test_protected_tokens_count_is_exact():
    s = _rand((3, 101), 16)
    for pct in (0, 1, 5, 10, 50, 100):
        n = orc.ceil_pct(pct, 101)
        flags = orc.protected_tokens(s, n)
        assert flags.sum(1).tolist() == [n] * 3
        for b in range(3):
            if 0 < n < 101:
                assert s[b][flags[b] == 1].min() >= s[b][flags[b] == 0].max()


def test_ceil_pct_integer_ceiling():
    assert orc.ceil_pct(10, 140) == 14          # 0.1*140 in floating point would round up to 15
    assert orc.ceil_pct(10, 256) == 26
    assert orc.ceil_pct(5, 32760) == 1638
    assert orc.ceil_pct(5, 17856) == 893
    assert orc.ceil_pct(20, 17856) == 3572
    assert orc.ceil_pct(5, 49152) == 2458
    assert orc.ceil_pct(20, 384) == 77
    assert orc.ceil_pct(25, 256) == 64
    assert orc.ceil_pct(0, 999) == 0 and orc.ceil_pct(100, 999) == 999


def test_protected_blocks_lift():
    flags = np.zeros((1, 10), np.uint8); flags[0, [3, 9]] = 1
    assert orc.protected_blocks(flags, 4).tolist() == [[1, 0, 1]]
    assert orc.protected_blocks(np.zeros((2, 10), np.uint8), 4).tolist() == [[0, 0, 0]] * 2
    # at least n tokens per block: block 0 holds {0,1,3}, block 1 holds {5}, the 2-token tail block holds {8,9}
    flags = np.zeros((1, 10), np.uint8); flags[0, [0, 1, 3, 5, 8, 9]] = 1
    assert orc.protected_blocks(flags, 4, min_tokens=1).tolist() == [[1, 1, 1]]
    assert orc.protected_blocks(flags, 4, min_tokens=2).tolist() == [[1, 0, 1]]
    assert orc.protected_blocks(flags, 4, min_tokens=3).tolist() == [[1, 0, 0]]
    assert orc.protected_blocks(flags, 4, min_tokens=4).tolist() == [[0, 0, 0]]


def test_protected_blocks_by_sum():
    """Hand example: block sums 6 | 6 | 1.5 (two-token tail): the best block is block 0 (tie with block 1, lowest
    index first), the best two are blocks 0 and 1; a NaN block ranks last."""
    s = np.array([[1, 2, 3, 0, 6, 0, 0, 0, 1, 0.5]], np.float32)
    assert orc.protected_blocks_by_sum(s, 4, 1).tolist() == [[1, 0, 0]]
    assert orc.protected_blocks_by_sum(s, 4, 2).tolist() == [[1, 1, 0]]
    assert orc.protected_blocks_by_sum(s, 4, 3).tolist() == [[1, 1, 1]]
    s[0, 1] = np.nan
    assert orc.protected_blocks_by_sum(s, 4, 1).tolist() == [[0, 1, 0]]
    assert orc.protected_blocks_by_sum(s, 4, 2).tolist() == [[0, 1, 1]]
    # through the whole mask step: all tokens of the chosen blocks are flagged, their rows are dense
    bs = np.zeros((1, 1, 3, 3), np.float32); bs[0, 0] = np.eye(3)
    s = np.array([[1, 2, 3, 0, 6, 0, 0, 0, 1, 0.5]], np.float32)
    idx, cnt, ptok, pblk = orc.build_block_mask(bs, s, 1, 1, 4, 10, block_sum=True)
    assert pblk.tolist() == [[1, 0, 0]] and ptok.tolist() == [[1, 1, 1, 1, 0, 0, 0, 0, 0, 0]]
    assert cnt[0, 0].tolist() == [3, 1, 1] and idx[0, 0, 1].tolist() == [1, -1, -1]


# ------------------------------------------------------------------------------- pooling, scores
def test_block_mean_pool_closed_forms():
    B, H, N, d, blk = 1, 2, 11, 3, 4                                 # tail block of 3 tokens
    x = np.full((B, H, N, d), 2.5)
    np.testing.assert_allclose(orc.block_mean_pool(x, blk), 2.5)
    ramp = np.broadcast_to(np.arange(N, dtype=np.float64)[None, None, :, None], (B, H, N, d))
    p = orc.block_mean_pool(ramp, blk)
    np.testing.assert_allclose(p[0, 0, :, 0], [1.5, 5.5, 9.0])      # (0+1+2+3)/4, (4..7)/4, (8+9+10)/3
    x = _rand((B, H, N, d), 17)
    p = orc.block_mean_pool(x, blk)
    np.testing.assert_allclose(p[0, 1, 2], (x[0, 1, 8] + x[0, 1, 9] + x[0, 1, 10]) / 3.0, rtol=1e-14)


def test_block_scores_brute_force_not_transposed():
    B, H, N, d, blk = 1, 2, 10, 4, 4
    q, k = _rand((B, H, N, d), 18), _rand((B, H, N, d), 19)
    bs = orc.block_scores(q, k, blk)
    for h in range(H):
        for i in range(3):
            for j in range(3):
                qi = [sum(q[0, h, t, c] for t in range(i * 4, min(i * 4 + 4, N))) / (min(i * 4 + 4, N) - i * 4) for c in range(d)]
                kj = [sum(k[0, h, t, c] for t in range(j * 4, min(j * 4 + 4, N))) / (min(j * 4 + 4, N) - j * 4) for c in range(d)]
                want = sum(a * b for a, b in zip(qi, kj)) / math.sqrt(d)
                assert abs(bs[0, h, i, j] - want) < 1e-13
    assert not np.allclose(bs, np.swapaxes(bs, -1, -2))


# ------------------------------------------------------------------------------- Eq. 9 lists
def test_mask_invariants():
    B, H, N, d, blk = 2, 3, 150, 8, 16                                # 10 blocks, tail of 6
    NB = 10
    q, k = _rand((B, H, N, d), 20), _rand((B, H, N, d), 21)
    bs = orc.block_scores(q, k, blk)
    s = _rand((B, N), 22)
    k_keep, n_prot = 3, 8
    idx, cnt, ptok, pblk = orc.build_block_mask(bs, s, n_prot, k_keep, blk, N)
    assert ptok.sum(1).tolist() == [n_prot] * B
    for b in range(B):
        for h in range(H):
            for i in range(NB):
                c = cnt[b, h, i]
                cols = idx[b, h, i, :c]
                assert c == (NB if pblk[b, i] else k_keep)             # Eq. 9 rows; exact budget elsewhere
                assert (np.diff(cols) > 0).all() and cols.min() >= 0 and cols.max() < NB
                assert (idx[b, h, i, c:] == -1).all()
                if not pblk[b, i]:
                    kept = set(cols.tolist())
                    lo = min(bs[b, h, i, j] for j in kept)
                    hi = max(bs[b, h, i, j] for j in range(NB) if j not in kept)
                    assert lo >= hi
    # token-level Eq. 9 mask is contained in the block mask
    for b in range(B):
        for t in np.nonzero(ptok[b])[0]:
            assert (cnt[b, :, t // blk] == NB).all()
    # k_keep = NB and n_protect = N both give the full mask
    for args in ((0, NB), (N, 1)):
        _, cnt2, _, _ = orc.build_block_mask(bs, s, args[0], args[1], blk, N)
        assert (cnt2 == NB).all()
    # column protection: every protected key block appears in every row
    idx3, cnt3, _, pblk3 = orc.build_block_mask(bs, s, n_prot, k_keep, blk, N, True, True)
    for b in range(B):
        for j in np.nonzero(pblk3[b])[0]:
            for h in range(H):
                for i in range(NB):
                    assert j in idx3[b, h, i, : cnt3[b, h, i]]


def test_topk_blocks_ties_lowest_index():
    bs = np.zeros((1, 1, 2, 6)); bs[0, 0, 1] = [1, 3, 3, 0, 3, 1]
    keep = orc.topk_blocks(bs, 2)
    assert keep[0, 0, 0].tolist() == [1, 1, 0, 0, 0, 0]
    assert keep[0, 0, 1].tolist() == [0, 1, 1, 0, 0, 0]


# ------------------------------------------------------------------------------- Eq. 10 / 11
def _additive_mask_attention(q, k, v, keep, blk, scale):
    """Eq. 6-7 written the other way: full logits plus a 0 / -inf matrix, then softmax."""
    N = q.shape[0]
    M = np.full((N, N), -np.inf)
    nb = keep.shape[0]
    for i in range(nb):
        for j in range(nb):
            if keep[i, j]:
                M[i * blk:(i + 1) * blk, j * blk:(j + 1) * blk] = 0.0
    s = q @ k.T * scale + M
    p = torch.softmax(torch.from_numpy(s), dim=-1).numpy()
    return p @ v


def test_masked_attention_vs_additive_mask_and_dense():
    B, H, N, d, blk = 1, 2, 45, 8, 8                                  # 6 blocks, tail of 5
    q, k, v = _rand((B, H, N, d), 23), _rand((B, H, N, d), 24), _rand((B, H, N, d), 25)
    bs = orc.block_scores(q, k, blk)
    s = _rand((B, N), 26)
    idx, cnt, ptok, pblk = orc.build_block_mask(bs, s, 3, 2, blk, N)
    O, lse = orc.masked_attention(q, k, v, idx, cnt, blk)
    dense, dense_lse = orc.dense_attention(q, k, v)
    for h in range(H):
        keep = np.zeros((6, 6), np.uint8)
        for i in range(6):
            keep[i, idx[0, h, i, : cnt[0, h, i]]] = 1
        want = _additive_mask_attention(q[0, h], k[0, h], v[0, h], keep, blk, 1 / math.sqrt(d))
        np.testing.assert_allclose(O[0, h], want, rtol=1e-11, atol=1e-12)
        # Eq. 11: rows of protected blocks are dense rows; some other row differs from dense
        for i in range(6):
            rows = slice(i * blk, min((i + 1) * blk, N))
            if pblk[0, i]:
                np.testing.assert_allclose(O[0, h, rows], dense[0, h, rows], rtol=1e-12, atol=1e-13)
                np.testing.assert_allclose(lse[0, h, rows], dense_lse[0, h, rows], rtol=1e-12)
            else:
                assert np.abs(O[0, h, rows] - dense[0, h, rows]).max() > 1e-6
    assert pblk.sum() >= 1 and pblk.sum() < 6
    # keep-all lists == dense attention == library attention
    idx_all, cnt_all, _, _ = orc.build_block_mask(bs, s, 0, 6, blk, N)
    O_all, lse_all = orc.masked_attention(q, k, v, idx_all, cnt_all, blk)
    np.testing.assert_allclose(O_all, dense, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lse_all, dense_lse, rtol=1e-12)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v)).numpy()
    np.testing.assert_allclose(O_all, ref, rtol=1e-10, atol=1e-12)
    # all tokens protected == dense
    idx_p, cnt_p, _, _ = orc.build_block_mask(bs, s, N, 1, blk, N)
    O_p, _ = orc.masked_attention(q, k, v, idx_p, cnt_p, blk)
    np.testing.assert_allclose(O_p, dense, rtol=1e-12, atol=1e-13)


def test_masked_attention_golden_closed_form():
    g = _golden()
    q = np.array([[1.0]]); k = np.array([[0.0], [math.log(3.0)], [math.log(4.0)]]); v = np.array([[8.0], [16.0], [24.0]])
    o, lse = orc.masked_attention_rows(q, k, v, [0, 1], 1, scale=1.0)
    assert abs(o[0, 0] - g["masked_out"]) < 1e-13 and abs(lse[0] - g["masked_lse"]) < 1e-13
    o, lse = orc.masked_attention_rows(q, k, v, [0, 1, 2], 1, scale=1.0)
    assert abs(o[0, 0] - g["dense_out"]) < 1e-13 and abs(lse[0] - g["dense_lse"]) < 1e-13


def test_masked_attention_brute_force_single_row():
    N, d, blk = 13, 3, 4
    q, k, v = _rand((N, d), 27), _rand((N, d), 28), _rand((N, d), 29)
    cols = [0, 3]                                                     # block 3 is the 1-token tail
    o, lse = orc.masked_attention_rows(q[4:8], k, v, cols, blk)
    keys = [0, 1, 2, 3, 12]
    for r in range(4):
        logits = [sum(q[4 + r, t] * k[j, t] for t in range(d)) / math.sqrt(d) for j in keys]
        z = sum(math.exp(x) for x in logits)
        for t in range(d):
            want = sum(math.exp(x) / z * v[j, t] for x, j in zip(logits, keys))
            assert abs(o[r, t] - want) < 1e-13
        assert abs(lse[r] - math.log(z)) < 1e-13


def test_token_exact_protection_is_eq9_on_tokens():
    """Eq. 9 written literally on tokens: 0 where the query is protected or the pair is in S, -inf elsewhere."""
    B, H, N, d, blk = 1, 2, 45, 8, 8
    q, k, v = _rand((B, H, N, d), 31), _rand((B, H, N, d), 32), _rand((B, H, N, d), 33)
    bs = orc.block_scores(q, k, blk)
    s = _rand((B, N), 34)
    n_protect = 4
    idx, cnt, ptok, pblk = orc.build_block_mask(bs, s, n_protect, 2, blk, N, protect_rows=False)
    assert (cnt == 2).all()                                            # base pattern only
    O, lse = orc.protected_attention_token_exact(q, k, v, idx, cnt, ptok, blk)
    dense, dense_lse = orc.dense_attention(q, k, v)
    sparse, _ = orc.masked_attention(q, k, v, idx, cnt, blk)
    for h in range(H):
        M = np.full((N, N), -np.inf)
        for i in range(6):
            for j in idx[0, h, i, : cnt[0, h, i]]:
                M[i * blk:(i + 1) * blk, j * blk:(j + 1) * blk] = 0.0
        M[ptok[0] == 1, :] = 0.0
        logits = q[0, h] @ k[0, h].T / math.sqrt(d) + M
        want = torch.softmax(torch.from_numpy(logits), dim=-1).numpy() @ v[0, h]
        np.testing.assert_allclose(O[0, h], want, rtol=1e-11, atol=1e-12)
        prot = ptok[0] == 1
        np.testing.assert_allclose(O[0, h, prot], dense[0, h, prot], rtol=1e-12, atol=1e-13)      # Eq. 11, first case
        np.testing.assert_allclose(lse[0, h, prot], dense_lse[0, h, prot], rtol=1e-12)
        np.testing.assert_allclose(O[0, h, ~prot], sparse[0, h, ~prot], rtol=1e-12, atol=1e-13)   # Eq. 11, second case
    assert ptok.sum() == n_protect


# ------------------------------------------------------------------------------- Eq. 12-15
def test_cache_indicators_golden_and_closed_forms():
    g = {}
    with open(os.path.join(os.path.dirname(GOLDEN), "cache_indicators_example.txt")) as f:
        for line in f:
            if not line.startswith("#") and line.strip():
                k, v = line.split()
                g[k] = float(v)
    r = orc.cache_indicators([[1, -2], [3, 4]], [[1, 0], [0, 4]], [[2, 2]], [[1, 3]], prot_tok=[0, 1],
                             s_cur=[1, 0], s_anchor=[1, 1], eps=0.0)
    for k in ("dv", "da", "dp", "ds", "dsync"):
        assert abs(r[k] - g[k]) < 1e-15, k
    assert r["reuse"] == bool(g["reuse"])
    # identical features and parallel saliency maps: nothing changed, reuse
    y = _rand((7, 4), 41); a = _rand((3, 4), 42); s = np.abs(_rand((7,), 43))
    r = orc.cache_indicators(y, y, a, a, prot_tok=[1, 0, 0, 1, 0, 0, 0], s_cur=s, s_anchor=3.0 * s, eps=0.0)
    assert r["dv"] == 0 and r["da"] == 0 and r["dp"] == 0 and abs(r["ds"]) < 1e-15 and r["reuse"]
    # cache of zeros: relative change 1; orthogonal saliency maps: drift 1; scale invariance of the ratios
    r = orc.cache_indicators(y, 0 * y, a, 0 * a, prot_tok=[0, 1, 0, 0, 0, 0, 0], s_cur=[1, 0, 0, 0, 0, 0, 0],
                             s_anchor=[0, 1, 0, 0, 0, 0, 0], eps=0.0)
    assert abs(r["dv"] - 1) < 1e-15 and abs(r["da"] - 1) < 1e-15 and abs(r["dp"] - 1) < 1e-15 and abs(r["ds"] - 1) < 1e-15
    yh = y + 0.1 * _rand((7, 4), 44)
    r1 = orc.cache_indicators(y, yh, a, a, eps=0.0)
    r2 = orc.cache_indicators(5 * y, 5 * yh, a, a, eps=0.0)
    assert abs(r1["dv"] - r2["dv"]) < 1e-15
    # Eq. 15 is a weighted maximum: each term can be the binding one
    assert orc.cache_indicators(y, yh, a, a + 10, eps=0.0)["dsync"] == orc.cache_indicators(y, yh, a, a + 10, eps=0.0)["da"]
    r = orc.cache_indicators(y, y, a, a, s_cur=[1, 0, 0, 0, 0, 0, 0], s_anchor=[0, 1, 0, 0, 0, 0, 0], lambda_s=0.1, eps=0.0)
    assert abs(r["dsync"] - 0.1) < 1e-15 and r["reuse"]            # 0.1 * 1 < tau = 0.2
