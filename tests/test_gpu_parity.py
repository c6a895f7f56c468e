"""GPU parity: every call of the C ABI against the fp64 CPU oracle on the same seeded inputs.

Bars: integer outputs (flags, lists, counts) bit-exact given the same fp32 score tensors.
bf16 attention outputs O: relative-L2 5e-3 and max-abs 1e-2, the latter scaled by |value| above 1 (the bf16
grid itself is coarser than 1e-2 there).  fp32 log-sum-exps: max-abs 1e-3, unscaled.  fp32 response scores
(Eq. 2): every element within 1e-3 of its own value (plus 1e-6 of the largest score), so that a few wrong
columns cannot hide in a norm.
"""
import numpy as np
import pytest
import torch

from oracle import avsa_oracle as orc
from paper_2608_15522_b200 import binding as av
from paper_2608_15522_b200 import workloads as wl
from parity_bars import close_lse as _close_lse, close_o as _close, close_scores as _close_scores, np64 as _np64

pytestmark = pytest.mark.gpu

def _status_ok(ws):
    code, detail = av.avsa_read_status(ws)
    assert code == av.AVSA_OK, f"device status {code} {av.status_string(code)} detail {detail}"


def _oracle_mask(w, q, k, scores64, n_protect, k_keep, flags=av.AVSA_PROTECT_ROWS):
    """Oracle block scores (rounded to fp32, the tensor both sides select from) and its lists."""
    bs32 = orc.block_scores(_np64(q), _np64(k), w.blk).astype(np.float32)
    s32 = scores64.astype(np.float32)
    idx, cnt, ptok, pblk = orc.build_block_mask(bs32, s32, n_protect, k_keep, w.blk, w.n_video,
                                                bool(flags & av.AVSA_PROTECT_ROWS), bool(flags & av.AVSA_PROTECT_COLS))
    return bs32, s32, idx, cnt, ptok, pblk


def _oracle_scores(w, seed):
    qa, kc, vc = wl.make_cross_qkv(w, seed)
    o, lse, A = orc.cross_attention(_np64(qa), _np64(kc), _np64(vc))
    s = orc.column_scores(A, gamma=1.0 / (w.H * w.n_audio))
    return (qa, kc, vc), o, lse, s


# ------------------------------------------------------------------------------------------- mask
@pytest.mark.parametrize("name,flags", [("tiny", 1), ("small128", 1), ("medium128", 1), ("medium128", 3)])
def test_mask_lists_bit_exact_given_oracle_scores(name, flags):
    w = wl.WORKLOADS[name]
    q, k, _ = wl.make_self_qkv(w, 0)
    _, _, _, s64 = _oracle_scores(w, 0)
    n_protect = orc.ceil_pct(w.protect_pct, w.n_video)
    k_keep = max(1, orc.ceil_pct(w.keep_pct, w.n_blocks))
    assert n_protect == av.avsa_count_from_percent(w.protect_pct, w.n_video)
    assert k_keep == max(1, av.avsa_count_from_percent(w.keep_pct, w.n_blocks))
    bs32, s32, idx, cnt, ptok, pblk = _oracle_mask(w, q, k, s64, n_protect, k_keep, flags)
    out = av.avsa_build_block_mask(None, None, torch.from_numpy(s32).cuda(), n_protect, k_keep, w.blk,
                                   flags=flags | av.AVSA_USE_GIVEN_BLOCK_SCORES,
                                   block_scores=torch.from_numpy(bs32).cuda(), shape=(w.B, w.H, w.n_video, w.d))
    _status_ok(out["ws"])
    assert np.array_equal(out["prot_tok"].cpu().numpy(), ptok)
    assert np.array_equal(out["prot_blk"].cpu().numpy(), pblk)
    assert np.array_equal(out["col_cnt"].cpu().numpy(), cnt)
    assert np.array_equal(out["col_idx"].cpu().numpy(), idx)


@pytest.mark.parametrize("name,min_tokens", [("tiny", 3), ("medium128", 2), ("medium128", 16), ("medium128", 128)])
def test_mask_min_tokens_per_block_bit_exact(name, min_tokens):
    """A block counts as protected only from `min_tokens` protected tokens on (flag bits 8-15)."""
    w = wl.WORKLOADS[name]
    _, _, _, s64 = _oracle_scores(w, 0)
    q, k, _ = wl.make_self_qkv(w, 0)
    n_protect = orc.ceil_pct(w.protect_pct, w.n_video)
    k_keep = max(1, orc.ceil_pct(w.keep_pct, w.n_blocks))
    bs32 = orc.block_scores(_np64(q), _np64(k), w.blk).astype(np.float32)
    s32 = s64.astype(np.float32)
    idx, cnt, ptok, pblk = orc.build_block_mask(bs32, s32, n_protect, k_keep, w.blk, w.n_video, True, False,
                                                min_tokens=min_tokens)
    any_blk = orc.protected_blocks(ptok, w.blk)
    if name == "medium128" and min_tokens >= 16:
        assert pblk.sum() < any_blk.sum()      # the threshold bites on these inputs
    out = av.avsa_build_block_mask(None, None, torch.from_numpy(s32).cuda(), n_protect, k_keep, w.blk,
                                   flags=av.AVSA_PROTECT_ROWS | av.AVSA_USE_GIVEN_BLOCK_SCORES |
                                   av.AVSA_MIN_TOKENS_PER_BLOCK(min_tokens),
                                   block_scores=torch.from_numpy(bs32).cuda(), shape=(w.B, w.H, w.n_video, w.d))
    _status_ok(out["ws"])
    assert np.array_equal(out["prot_tok"].cpu().numpy(), ptok)
    assert np.array_equal(out["prot_blk"].cpu().numpy(), pblk)
    assert np.array_equal(out["col_cnt"].cpu().numpy(), cnt)
    assert np.array_equal(out["col_idx"].cpu().numpy(), idx)


@pytest.mark.parametrize("name,n_blocks,extra", [("tiny", 1, 0), ("medium128", 3, 0), ("medium128", 5, 2),
                                                 ("medium128", 0, 0), ("medium128", 17, 0)])
def test_mask_block_sum_protection_bit_exact(name, n_blocks, extra):
    """Protected blocks = the n blocks with the largest summed response (flag AVSA_PROTECT_BLOCK_SUM), also with
    key-column protection on top (extra = AVSA_PROTECT_COLS).  Block flags, token flags and lists bit-exact."""
    w = wl.WORKLOADS[name]
    _, _, _, s64 = _oracle_scores(w, 0)
    q, k, _ = wl.make_self_qkv(w, 0)
    k_keep = max(1, orc.ceil_pct(w.keep_pct, w.n_blocks))
    bs32 = orc.block_scores(_np64(q), _np64(k), w.blk).astype(np.float32)
    s32 = s64.astype(np.float32)
    s32[:, 5] = np.nan                                   # a NaN score poisons its block's sum: that block ranks last
    idx, cnt, ptok, pblk = orc.build_block_mask(bs32, s32, n_blocks, k_keep, w.blk, w.n_video, True, bool(extra),
                                                block_sum=True)
    assert pblk.sum() == n_blocks * w.B and (n_blocks == w.n_blocks or pblk[:, 0].sum() == 0)
    out = av.avsa_build_block_mask(None, None, torch.from_numpy(s32).cuda(), n_blocks, k_keep, w.blk,
                                   flags=av.AVSA_PROTECT_ROWS | extra | av.AVSA_USE_GIVEN_BLOCK_SCORES |
                                   av.AVSA_PROTECT_BLOCK_SUM,
                                   block_scores=torch.from_numpy(bs32).cuda(), shape=(w.B, w.H, w.n_video, w.d))
    _status_ok(out["ws"])
    assert np.array_equal(out["prot_blk"].cpu().numpy(), pblk)
    assert np.array_equal(out["prot_tok"].cpu().numpy(), ptok)
    assert np.array_equal(out["col_cnt"].cpu().numpy(), cnt)
    assert np.array_equal(out["col_idx"].cpu().numpy(), idx)


def test_mask_ties_nan_and_signed_zero_bit_exact():
    B, H, N, d, blk = 2, 2, 64 * 37 + 5, 64, 64
    NB = (N + blk - 1) // blk
    rng = np.random.default_rng(3)
    bs = rng.integers(-2, 3, size=(B, H, NB, NB)).astype(np.float32)          # heavy ties
    bs[0, 0, 1, :] = 0.0
    bs[0, 0, 2, ::2] = -0.0
    bs[0, 1, 3, 5] = np.nan
    bs[1, 0, 4, :] = np.nan
    bs[1, 1, 5, 7] = np.inf
    bs[1, 1, 5, 9] = -np.inf
    s = rng.integers(0, 4, size=(B, N)).astype(np.float32)
    s[0, 10] = np.nan
    s[1, ::3] = -0.0
    for n_protect, k_keep in ((0, 1), (7, 5), (200, NB), (N, 3), (1, NB - 1)):
        idx, cnt, ptok, pblk = orc.build_block_mask(bs, s, n_protect, k_keep, blk, N)
        out = av.avsa_build_block_mask(None, None, torch.from_numpy(s).cuda(), n_protect, k_keep, blk,
                                       flags=av.AVSA_PROTECT_ROWS | av.AVSA_USE_GIVEN_BLOCK_SCORES,
                                       block_scores=torch.from_numpy(bs).cuda(), shape=(B, H, N, d))
        _status_ok(out["ws"])
        assert np.array_equal(out["prot_tok"].cpu().numpy(), ptok), (n_protect, k_keep)
        assert np.array_equal(out["prot_blk"].cpu().numpy(), pblk), (n_protect, k_keep)
        assert np.array_equal(out["col_cnt"].cpu().numpy(), cnt), (n_protect, k_keep)
        assert np.array_equal(out["col_idx"].cpu().numpy(), idx), (n_protect, k_keep)


def test_mask_long_sequence_beyond_the_shared_memory_key_cache():
    """N above 57344 tokens: the token select re-reads global memory instead of staging keys on chip."""
    B, H, N, d, blk = 2, 1, 60000 + 77, 128, 128
    NB = (N + blk - 1) // blk
    rng = np.random.default_rng(9)
    bs = rng.standard_normal((B, H, NB, NB)).astype(np.float32)
    s = np.round(rng.standard_normal((B, N)) * 50).astype(np.float32) / 50      # many exact ties
    n_protect, k_keep = 3001, 40
    idx, cnt, ptok, pblk = orc.build_block_mask(bs, s, n_protect, k_keep, blk, N)
    out = av.avsa_build_block_mask(None, None, torch.from_numpy(s).cuda(), n_protect, k_keep, blk,
                                   flags=av.AVSA_PROTECT_ROWS | av.AVSA_USE_GIVEN_BLOCK_SCORES,
                                   block_scores=torch.from_numpy(bs).cuda(), shape=(B, H, N, d))
    _status_ok(out["ws"])
    assert np.array_equal(out["prot_tok"].cpu().numpy(), ptok)
    assert np.array_equal(out["prot_blk"].cpu().numpy(), pblk)
    assert np.array_equal(out["col_cnt"].cpu().numpy(), cnt)
    assert np.array_equal(out["col_idx"].cpu().numpy(), idx)


@pytest.mark.parametrize("name", ["tiny", "small128", "medium128"])
def test_block_scores_and_selection_from_pooled_qk(name):
    w = wl.WORKLOADS[name]
    q, k, _ = wl.make_self_qkv(w, 1)
    _, _, _, s64 = _oracle_scores(w, 1)
    n_protect = orc.ceil_pct(w.protect_pct, w.n_video)
    k_keep = max(1, orc.ceil_pct(w.keep_pct, w.n_blocks))
    s32 = s64.astype(np.float32)
    out = av.avsa_build_block_mask(q.cuda(), k.cuda(), torch.from_numpy(s32).cuda(), n_protect, k_keep, w.blk)
    _status_ok(out["ws"])
    want = orc.block_scores(_np64(q), _np64(k), w.blk)
    got = out["block_scores"].cpu().numpy()
    assert np.abs(got - want).max() <= 1e-4 * max(1.0, np.abs(want).max())
    # the lists are exactly the oracle's when it selects from the very tensor the GPU produced
    idx, cnt, ptok, pblk = orc.build_block_mask(got, s32, n_protect, k_keep, w.blk, w.n_video)
    assert np.array_equal(out["col_idx"].cpu().numpy(), idx)
    assert np.array_equal(out["col_cnt"].cpu().numpy(), cnt)
    assert np.array_equal(out["prot_tok"].cpu().numpy(), ptok)
    # and a valid top-k of the oracle's own fp64 scores up to the fp32 rounding of the scores
    gidx, gcnt = out["col_idx"].cpu().numpy(), out["col_cnt"].cpu().numpy()
    tol = 2e-4 * max(1.0, np.abs(want).max())
    for b in range(w.B):
        for h in range(w.H):
            for i in range(w.n_blocks):
                if pblk[b, i] or k_keep >= w.n_blocks:
                    continue
                kept = gidx[b, h, i, : gcnt[b, h, i]]
                rest = np.setdiff1d(np.arange(w.n_blocks), kept)
                assert want[b, h, i, kept].min() >= want[b, h, i, rest].max() - tol


@pytest.mark.parametrize("d,nb,tail", [(128, 520, 5), (64, 300, 17), (128, 33, 0)])
def test_block_scores_and_lists_long_rows(d, nb, tail):
    """Rows of more than 256 and more than 512 key blocks (more keys per lane in the select, larger strips in shared
    memory), a ragged last block, and a block count that is no multiple of the 16-row strip: pooled block scores
    against the oracle, lists bit-exact given those scores."""
    blk = d
    N = blk * (nb - 1) + (tail if tail else blk)
    B, H = 1, 2
    g = torch.Generator().manual_seed(nb)
    q = torch.randn((B, H, N, d), generator=g).bfloat16()
    k = (torch.randn((B, H, N, d), generator=g) + 0.5).bfloat16()
    s = torch.rand((B, N), generator=g)
    n_protect, k_keep = N // 50, max(1, nb // 5)
    out = av.avsa_build_block_mask(q.cuda(), k.cuda(), s.cuda(), n_protect, k_keep, blk)
    _status_ok(out["ws"])
    got = out["block_scores"].cpu().numpy()
    want = orc.block_scores(_np64(q), _np64(k), blk)
    assert got.shape == (B, H, nb, nb)
    assert np.abs(got - want).max() <= 1e-4 * max(1.0, np.abs(want).max())
    idx, cnt, ptok, pblk = orc.build_block_mask(got, s.numpy(), n_protect, k_keep, blk, N)
    assert np.array_equal(out["col_cnt"].cpu().numpy(), cnt)
    assert np.array_equal(out["col_idx"].cpu().numpy(), idx)
    assert np.array_equal(out["prot_tok"].cpu().numpy(), ptok) and np.array_equal(out["prot_blk"].cpu().numpy(), pblk)


# ------------------------------------------------------------------------------------------- sparse attention
def _run_sparse_case(w, seed, idx, cnt, want_lse=True):
    q, k, v = wl.make_self_qkv(w, seed)
    o, lse, ws = av.avsa_sparse_self_attn(q.cuda(), k.cuda(), v.cuda(), torch.from_numpy(idx).cuda(),
                                          torch.from_numpy(cnt).cuda(), w.blk, want_lse=want_lse)
    _status_ok(ws)
    # the workloads' logits stay within a few units of each row's first-tile maximum: every item must come from
    # the fast kernel (the growing-maxima tests cover the recomputation path)
    assert av.avsa_redo_count(ws) == 0
    want_o, want_l = orc.masked_attention(_np64(q), _np64(k), _np64(v), idx, cnt, w.blk)
    _close(_np64(o), want_o, f"{w.name} O")
    if want_lse:
        _close_lse(_np64(lse), want_l, f"{w.name} lse")
    return _np64(o), want_o


@pytest.mark.parametrize("name", ["tiny", "small128", "medium128"])
def test_sparse_attention_matches_oracle_under_protected_mask(name):
    w = wl.WORKLOADS[name]
    q, k, _ = wl.make_self_qkv(w, 0)
    _, _, _, s64 = _oracle_scores(w, 0)
    n_protect = orc.ceil_pct(w.protect_pct, w.n_video)
    k_keep = max(1, orc.ceil_pct(w.keep_pct, w.n_blocks))
    _, _, idx, cnt, _, pblk = _oracle_mask(w, q, k, s64, n_protect, k_keep)
    assert 0 < pblk.sum() < pblk.size or name == "small128"
    _run_sparse_case(w, 0, idx, cnt)


@pytest.mark.parametrize("name", ["tiny", "small128", "medium128"])
def test_sparse_attention_keep_all_is_dense(name):
    w = wl.WORKLOADS[name]
    NB = w.n_blocks
    idx = np.broadcast_to(np.arange(NB, dtype=np.int32), (w.B, w.H, NB, NB)).copy()
    cnt = np.full((w.B, w.H, NB), NB, np.int32)
    got, _ = _run_sparse_case(w, 2, idx, cnt)
    q, k, v = wl.make_self_qkv(w, 2)
    dense, _ = orc.dense_attention(_np64(q), _np64(k), _np64(v))
    _close(got, dense, f"{name} keep-all vs dense")


def test_sparse_attention_single_and_odd_counts():
    """Lists of 1, 2 and 3 entries, and the last (ragged) key block alone."""
    w = wl.WORKLOADS["medium128"]
    NB = w.n_blocks
    idx = np.full((w.B, w.H, NB, NB), -1, np.int32)
    cnt = np.zeros((w.B, w.H, NB), np.int32)
    rng = np.random.default_rng(5)
    for b in range(w.B):
        for h in range(w.H):
            for i in range(NB):
                c = 1 + (i % 3)
                cols = np.sort(rng.choice(NB, size=c, replace=False))
                if i == 4:
                    cols = np.array([NB - 1])
                idx[b, h, i, :c] = cols
                cnt[b, h, i] = len(cols)
    _run_sparse_case(w, 3, idx, cnt)


@pytest.mark.parametrize("step,expect_redo,heads", [(1.0, False, 4), (16.0, True, 4), (16.0, True, 12)])
def test_sparse_attention_row_maxima_growing_along_the_key_axis(step, expect_redo, heads):
    """Logits that grow from key block to key block.  The fast kernel keeps the first tile's row maximum
    as its reference: a moderate growth stays inside its headroom, a steep one makes it hand the work item
    to the exact-rescaling kernel (listed behind the status record in the workspace).  Both must match
    the oracle; in the steep case items must actually have been handed over (with 12 heads more of them than
    the exact kernel has CTAs, so that its CTAs take several items each)."""
    import dataclasses
    w = dataclasses.replace(wl.WORKLOADS["medium128"], H=heads)
    q, k, v = wl.make_self_qkv(w, 6)
    NB = w.n_blocks
    u = 1.0 / np.sqrt(w.d)
    q = (q.float() + 8.0 * u).to(torch.bfloat16)
    ramp = torch.arange(w.n_video, dtype=torch.float32).div(w.blk, rounding_mode="floor") * step
    k = (k.float() + (ramp * u).view(1, 1, -1, 1)).to(torch.bfloat16)
    rng = np.random.default_rng(8)
    idx = np.full((w.B, w.H, NB, NB), -1, np.int32)
    cnt = np.zeros((w.B, w.H, NB), np.int32)
    for b in range(w.B):
        for h in range(w.H):
            for i in range(NB):
                c = NB if i % 4 == 0 else 1 + int(rng.integers(NB))
                cols = np.sort(rng.choice(NB, size=c, replace=False))
                idx[b, h, i, :c] = cols
                cnt[b, h, i] = c
    o, lse, ws = av.avsa_sparse_self_attn(q.cuda(), k.cuda(), v.cuda(), torch.from_numpy(idx).cuda(),
                                          torch.from_numpy(cnt).cuda(), w.blk, want_lse=True)
    _status_ok(ws)
    want_o, want_l = orc.masked_attention(_np64(q), _np64(k), _np64(v), idx, cnt, w.blk)
    _close(_np64(o), want_o, "growing maxima O")
    _close_lse(_np64(lse), want_l, "growing maxima lse")
    n_redo, items = av.avsa_sparse_self_attn_redo_items(ws)
    assert (n_redo > 0) == expect_redo
    if heads > 4:
        assert n_redo > 2 * 148
    if expect_redo:
        assert len(set(items.tolist())) == n_redo and items.min() >= 0 and items.max() < w.B * w.H * NB
        # items with a single key block never outgrow their reference
        assert np.all(cnt.reshape(-1)[items] > 1)


def test_sparse_attention_is_reproducible_over_repeated_launches():
    """Same inputs, 25 launches into fresh outputs: every result is bit-identical (the accumulation order is
    fixed by the lists, so any difference would be a race between the pipeline's stages)."""
    w = wl.WORKLOADS["medium128"]
    q, k, v = (t.cuda() for t in wl.make_self_qkv(w, 9))
    NB = w.n_blocks
    rng = np.random.default_rng(11)
    idx = np.full((w.B, w.H, NB, NB), -1, np.int32)
    cnt = np.zeros((w.B, w.H, NB), np.int32)
    for b in range(w.B):
        for h in range(w.H):
            for i in range(NB):
                c = 1 + int(rng.integers(NB))
                idx[b, h, i, :c] = np.sort(rng.choice(NB, size=c, replace=False))
                cnt[b, h, i] = c
    idx_d, cnt_d = torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda()
    first, first_lse, ws = av.avsa_sparse_self_attn(q, k, v, idx_d, cnt_d, w.blk, want_lse=True)
    _status_ok(ws)
    for _ in range(24):
        o, lse, ws = av.avsa_sparse_self_attn(q, k, v, idx_d, cnt_d, w.blk, want_lse=True)
        assert torch.equal(o, first) and torch.equal(lse, first_lse)
    _status_ok(ws)
    want_o, want_l = orc.masked_attention(_np64(q), _np64(k), _np64(v), idx, cnt, w.blk)
    _close(_np64(first), want_o, "random lists O")
    _close_lse(_np64(first_lse), want_l, "random lists lse")


def test_sparse_attention_strided_bnhd_layout():
    w = wl.WORKLOADS["small128"]
    q, k, v = wl.make_self_qkv(w, 4)
    NB = w.n_blocks
    idx = np.broadcast_to(np.arange(NB, dtype=np.int32), (w.B, w.H, NB, NB)).copy()
    cnt = np.full((w.B, w.H, NB), NB, np.int32)
    # storage [B,N,H,d], viewed as [B,H,N,d]
    qs, ks, vs = (t.cuda().permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) for t in (q, k, v))
    assert not qs.is_contiguous()
    o, _, ws = av.avsa_sparse_self_attn(qs, ks, vs, torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda(), w.blk)
    _status_ok(ws)
    assert o.stride() == qs.stride()
    want, _ = orc.dense_attention(_np64(q), _np64(k), _np64(v))
    _close(_np64(o), want, "strided O")


@pytest.mark.parametrize("seed", range(8))
def test_sparse_attention_random_shapes_and_lists(seed):
    """Seeded random shapes (batch, heads, length incl. ragged tails and lengths below one block, both tile
    sizes) with random ascending lists of random length, against the oracle."""
    rng = np.random.default_rng(100 + seed)
    d = int(rng.choice([64, 128]))
    blk = d
    B, H = int(rng.integers(1, 4)), int(rng.integers(1, 6))
    N = int(rng.integers(1, 9 * blk))
    NB = (N + blk - 1) // blk
    g = torch.Generator().manual_seed(200 + seed)
    q, k, v = (torch.randn(B, H, N, d, generator=g).to(torch.bfloat16) for _ in range(3))
    idx = np.full((B, H, NB, NB), -1, np.int32)
    cnt = np.zeros((B, H, NB), np.int32)
    for b in range(B):
        for h in range(H):
            for i in range(NB):
                c = 1 + int(rng.integers(NB))
                idx[b, h, i, :c] = np.sort(rng.choice(NB, size=c, replace=False))
                cnt[b, h, i] = c
    o, lse, ws = av.avsa_sparse_self_attn(q.cuda(), k.cuda(), v.cuda(), torch.from_numpy(idx).cuda(),
                                          torch.from_numpy(cnt).cuda(), blk, want_lse=True)
    _status_ok(ws)
    assert av.avsa_redo_count(ws) == 0             # unit-variance logits: nothing outgrows its reference
    want_o, want_l = orc.masked_attention(_np64(q), _np64(k), _np64(v), idx, cnt, blk)
    _close(_np64(o), want_o, f"random shape B{B} H{H} N{N} d{d} O")
    _close_lse(_np64(lse), want_l, f"random shape B{B} H{H} N{N} d{d} lse")


def test_sparse_attention_rows_not_32_byte_aligned():
    """Rows 272 bytes apart (d padded by 8 elements): 16-byte aligned, which is all the interface asks for (the
    tile loads and the staged tile store go through tensor maps).  Same result as the contiguous layout, bit for bit."""
    w = wl.WORKLOADS["medium128"]
    q, k, v = wl.make_self_qkv(w, 12)
    NB = w.n_blocks
    _, _, _, s64 = _oracle_scores(w, 0)
    n_protect = orc.ceil_pct(w.protect_pct, w.n_video)
    k_keep = max(1, orc.ceil_pct(w.keep_pct, NB))
    _, _, idx, cnt, _, _ = _oracle_mask(w, q, k, s64, n_protect, k_keep)

    def padded(t):
        buf = torch.zeros(t.shape[:-1] + (w.d + 8,), dtype=t.dtype, device="cuda")
        buf[..., : w.d] = t.cuda()
        return buf[..., : w.d]

    qp, kp, vp = padded(q), padded(k), padded(v)
    assert qp.stride(2) == w.d + 8 and qp.stride(3) == 1
    o, lse, ws = av.avsa_sparse_self_attn(qp, kp, vp, torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda(), w.blk,
                                          want_lse=True)
    _status_ok(ws)
    assert o.stride() == qp.stride()
    want_o, want_l = orc.masked_attention(_np64(q), _np64(k), _np64(v), idx, cnt, w.blk)
    _close(_np64(o), want_o, "padded rows O")
    _close_lse(_np64(lse), want_l, "padded rows lse")
    # and the contiguous layout gives the same numbers bit for bit
    o2, lse2, ws2 = av.avsa_sparse_self_attn(q.cuda(), k.cuda(), v.cuda(), torch.from_numpy(idx).cuda(),
                                             torch.from_numpy(cnt).cuda(), w.blk, want_lse=True)
    _status_ok(ws2)
    assert torch.equal(o2, o.contiguous()) and torch.equal(lse2, lse)


def test_sparse_attention_rejects_malformed_lists_without_touching_memory():
    w = wl.WORKLOADS["small128"]
    q, k, v = (t.cuda() for t in wl.make_self_qkv(w, 0))
    NB = w.n_blocks
    for bad in ([0, 0], [2, 1], [0, NB], [-1, 1]):
        idx = np.broadcast_to(np.arange(NB, dtype=np.int32), (w.B, w.H, NB, NB)).copy()
        cnt = np.full((w.B, w.H, NB), NB, np.int32)
        idx[0, 1, 2, :2] = bad
        cnt[0, 1, 2] = 2
        o, _, ws = av.avsa_sparse_self_attn(q, k, v, torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda(), w.blk)
        code, detail = av.avsa_read_status(ws)
        assert code == av.AVSA_ERR_BAD_MASK
        assert detail[1] == (0 * w.H + 1) * NB + 2
    cnt = np.zeros((w.B, w.H, NB), np.int32)
    o, _, ws = av.avsa_sparse_self_attn(q, k, v, torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda(), w.blk)
    assert av.avsa_read_status(ws)[0] == av.AVSA_ERR_BAD_MASK


def test_sparse_attention_skips_only_the_malformed_item_of_a_long_queue():
    """408 work items on 148 persistent CTAs, three of them malformed (bad count, descending entries, entry out
    of range): the status says BAD_MASK, the malformed items' rows are left untouched, every other row is right."""
    import dataclasses
    w = dataclasses.replace(wl.WORKLOADS["medium128"], H=12)
    q, k, v = wl.make_self_qkv(w, 13)
    NB = w.n_blocks
    rng = np.random.default_rng(14)
    idx = np.full((w.B, w.H, NB, NB), -1, np.int32)
    cnt = np.zeros((w.B, w.H, NB), np.int32)
    for b in range(w.B):
        for h in range(w.H):
            for i in range(NB):
                c = 1 + int(rng.integers(6))
                idx[b, h, i, :c] = np.sort(rng.choice(NB, size=c, replace=False))
                cnt[b, h, i] = c
    good_idx, good_cnt = idx.copy(), cnt.copy()
    bad_items = [(0, 3, 5), (1, 7, 0), (1, 11, 16)]
    cnt[0, 3, 5] = NB + 1
    idx[1, 7, 0, :2] = [4, 2]; cnt[1, 7, 0] = 2
    idx[1, 11, 16, :1] = [NB]; cnt[1, 11, 16] = 1
    o = torch.full((w.B, w.H, w.n_video, w.d), 7.0, dtype=torch.bfloat16, device="cuda")
    _, _, ws = av.avsa_sparse_self_attn(q.cuda(), k.cuda(), v.cuda(), torch.from_numpy(idx).cuda(),
                                        torch.from_numpy(cnt).cuda(), w.blk, o=o)
    code, detail = av.avsa_read_status(ws)
    assert code == av.AVSA_ERR_BAD_MASK
    assert detail[1] in [(b * w.H + h) * NB + i for b, h, i in bad_items]
    want, _ = orc.masked_attention(_np64(q), _np64(k), _np64(v), good_idx, good_cnt, w.blk)
    got = _np64(o)
    for b, h, i in bad_items:
        lo, hi = i * w.blk, min((i + 1) * w.blk, w.n_video)
        assert np.all(got[b, h, lo:hi] == 7.0)              # refused: nothing written
        want[b, h, lo:hi] = 7.0
    _close(got, want, "queue with malformed items")


# ------------------------------------------------------------------------------------------- cross attention
@pytest.mark.parametrize("name", ["tiny", "small128", "medium128"])
def test_cross_attention_outputs_and_scores(name):
    w = wl.WORKLOADS[name]
    (qa, kc, vc), want_o, want_lse, want_s = _oracle_scores(w, 0)
    gamma = 1.0 / (w.H * w.n_audio)
    o, lse, s, ws = av.avsa_cross_attn_scores(qa.cuda(), kc.cuda(), vc.cuda(), score_gamma=gamma)
    _status_ok(ws)
    assert av.avsa_redo_count(ws) == 0             # the planted boost (a few nats) stays inside the fast kernel's range
    _close(_np64(o), want_o, f"{name} cross O")
    _close_lse(_np64(lse), want_lse, f"{name} cross lse")
    got_s = _np64(s)
    assert abs(got_s.sum() - w.B) < 2e-3 * w.B                          # rows of Eq. 1 sum to one
    _close_scores(got_s, want_s, f"{name} scores (L1 norm)")
    # raw column mass (gamma = 1): every video token's score on its own, so that a wrong column cannot hide
    _, _, s_raw, _ = av.avsa_cross_attn_scores(qa.cuda(), kc.cuda(), vc.cuda(), score_gamma=1.0, want_o=False)
    _close_scores(_np64(s_raw), want_s * (w.H * w.n_audio), f"{name} scores (raw column mass)")
    # running blend (Eq. 4) and bit-for-bit reproducibility
    prev = torch.rand_like(s) * float(want_s.max())
    s2 = prev.clone()
    av.avsa_cross_attn_scores(qa.cuda(), kc.cuda(), vc.cuda(), scores=s2, score_beta=0.25, score_gamma=0.75 * gamma)
    torch.cuda.synchronize()
    want2 = 0.25 * _np64(prev) + 0.75 * want_s
    _close_scores(_np64(s2), want2, f"{name} blended scores (Eq. 4)")
    _, _, s3, _ = av.avsa_cross_attn_scores(qa.cuda(), kc.cuda(), vc.cuda(), score_gamma=gamma)
    assert torch.equal(s, s3)


def test_cross_attention_long_query_axis_two_chunks():
    """More than 256 queries: the column-sum pass splits the query axis in two."""
    w = wl.Workload("x", 1, 2, 128, 2, 9, 17, 300, 128, 50, 10, 1.0, ((0, 1, 1, 3, 2, 4),))
    (qa, kc, vc), want_o, want_lse, want_s = _oracle_scores(w, 7)
    o, lse, s, ws = av.avsa_cross_attn_scores(qa.cuda(), kc.cuda(), vc.cuda(), score_gamma=1.0 / (w.H * w.n_audio))
    _status_ok(ws)
    _close(_np64(o), want_o, "cross O")
    _close_lse(_np64(lse), want_lse, "cross lse")
    _close_scores(_np64(s), want_s, "scores, two query chunks")


@pytest.mark.parametrize("name", ["tiny", "small128", "medium128"])
def test_cross_attention_reverse_direction(name):
    """Video queries attending to audio keys (the other half of the bidirectional pair): outputs, LSE, and the
    audio-token saliency as column sums over the video queries (handled "analogously", Sec. 4.1)."""
    w = wl.WORKLOADS[name]
    qa, kc, vc = wl.make_cross_qkv(w, 3)
    q_video, k_audio, v_audio = kc, qa, wl.make_cross_qkv(w, 4)[0]          # roles swapped; fresh audio values
    want_o, want_lse, A = orc.cross_attention(_np64(q_video), _np64(k_audio), _np64(v_audio))
    gamma = 1.0 / (w.H * w.n_video)
    want_s = orc.column_scores(A, gamma=gamma)
    o, lse, s, ws = av.avsa_cross_attn_scores(q_video.cuda(), k_audio.cuda(), v_audio.cuda(), score_gamma=gamma)
    _status_ok(ws)
    _close(_np64(o), want_o, f"{name} reverse O")
    _close_lse(_np64(lse), want_lse, f"{name} reverse lse")
    got_s = _np64(s)
    assert got_s.shape == (w.B, w.n_audio)
    assert abs(got_s.sum() - w.B) < 2e-3 * w.B
    _close_scores(got_s, want_s, f"{name} reverse scores")
    _, _, s2, _ = av.avsa_cross_attn_scores(q_video.cuda(), k_audio.cuda(), v_audio.cuda(), score_gamma=gamma)
    assert torch.equal(s, s2)                                              # fixed summation order


@pytest.mark.parametrize("reverse", [False, True])
def test_cross_attention_row_maxima_growing_along_the_key_axis(reverse):
    """Pass 1 runs on the fast kernel too (key axis split across work items, or one item per query tile in the
    reverse direction): with logits that grow steeply from key block to key block its rows outgrow their
    first-tile reference and the exact-rescaling kernel must take the items over."""
    import dataclasses
    w = dataclasses.replace(wl.WORKLOADS["medium128"], H=12)      # forward: 24 query tiles -> key splits of 3 tiles
    qa, kc, vc = wl.make_cross_qkv(w, 3)
    if reverse:
        qa, kc, vc = kc, torch.cat([qa, qa, qa], dim=2), torch.cat([qa, qa, qa], dim=2).flip(2)   # 2070 queries, 216 keys
    u = 1.0 / np.sqrt(w.d)
    qa = (qa.float() + 8.0 * u).to(torch.bfloat16)
    nk = kc.shape[2]
    ramp = torch.arange(nk, dtype=torch.float32).div(w.blk, rounding_mode="floor") * (80.0 if reverse else 48.0)
    kc = (kc.float() + (ramp * u).view(1, 1, -1, 1)).to(torch.bfloat16)
    o, lse, _, ws = av.avsa_cross_attn_scores(qa.cuda(), kc.cuda(), vc.cuda(), want_scores=False)
    _status_ok(ws)
    assert av.avsa_redo_count(ws) > 0
    want_o, want_lse, _ = orc.cross_attention(_np64(qa), _np64(kc), _np64(vc))
    _close(_np64(o), want_o, "growing maxima cross O")
    _close_lse(_np64(lse), want_lse, "growing maxima cross lse")


def test_cross_attention_scores_need_one_short_axis():
    """Neither the queries nor the keys of a head fit on chip: the score pass is refused on the host."""
    q = torch.zeros((1, 1, 1024, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(av.AvsaError) as e:
        av.avsa_cross_attn_scores(q, q, q)
    assert e.value.status == av.AVSA_ERR_UNSUPPORTED
    o, lse, s, ws = av.avsa_cross_attn_scores(q, q, q, want_scores=False)  # outputs alone are fine
    _status_ok(ws)


# ------------------------------------------------------------------------------------------- whole path
def test_whole_path_tiny_matches_oracle():
    w = wl.WORKLOADS["tiny"]
    qa, kc, vc = (t.cuda() for t in wl.make_cross_qkv(w, 0))
    q, k, v = (t.cuda() for t in wl.make_self_qkv(w, 0))
    n_protect = av.avsa_count_from_percent(w.protect_pct, w.n_video)
    k_keep = av.avsa_count_from_percent(w.keep_pct, w.n_blocks)
    assert (n_protect, k_keep) == (26, 2)
    _, _, s, _ = av.avsa_cross_attn_scores(qa, kc, vc, score_gamma=1.0 / (w.H * w.n_audio))
    m = av.avsa_build_block_mask(q, k, s, n_protect, k_keep, w.blk)
    o, _, ws = av.avsa_sparse_self_attn(q, k, v, m["col_idx"], m["col_cnt"], w.blk)
    _status_ok(ws)
    assert av.avsa_redo_count(ws) == 0            # unit-variance logits never outgrow the first-tile reference
    # oracle end to end
    _, _, A = orc.cross_attention(_np64(qa), _np64(kc), _np64(vc))
    s64 = orc.column_scores(A, gamma=1.0 / (w.H * w.n_audio))
    bs64 = orc.block_scores(_np64(q), _np64(k), w.blk)
    idx, cnt, ptok, pblk = orc.build_block_mask(bs64, s64, n_protect, k_keep, w.blk, w.n_video)
    region = wl.region_mask(w, "cpu").numpy()
    assert (ptok[0].astype(bool) & region).sum() >= 24                    # the planted region is what gets protected
    # the planted margin makes the selections agree exactly between fp32/bf16 GPU scores and fp64 oracle
    assert np.array_equal(m["prot_blk"].cpu().numpy(), pblk)
    assert np.array_equal(m["col_cnt"].cpu().numpy(), cnt)
    assert np.array_equal(m["col_idx"].cpu().numpy(), idx)
    want, _ = orc.masked_attention(_np64(q), _np64(k), _np64(v), idx, cnt, w.blk)
    _close(_np64(o), want, "whole path O")


@pytest.mark.parametrize("name", ["tiny", "medium128"])
def test_whole_path_replays_from_a_cuda_graph(name):
    """The calls only enqueue work on the given stream (no allocation, no synchronisation, no host read of
    device data), so one layer-step can be captured into a CUDA graph once and replayed on new inputs.
    The replays must reproduce the eager results bit for bit, and the eager results are held to the oracle."""
    w = wl.WORKLOADS[name]
    n_protect = av.avsa_count_from_percent(w.protect_pct, w.n_video)
    k_keep = av.avsa_count_from_percent(w.keep_pct, w.n_blocks)
    gamma = 1.0 / (w.H * w.n_audio)

    def inputs(seed):
        return [t.cuda() for t in wl.make_cross_qkv(w, seed)] + [t.cuda() for t in wl.make_self_qkv(w, seed)]

    def eager(qa, kc, vc, q, k, v):
        _, _, s, _ = av.avsa_cross_attn_scores(qa, kc, vc, score_gamma=gamma, want_o=False)
        m = av.avsa_build_block_mask(q, k, s, n_protect, k_keep, w.blk)
        o, lse, ws = av.avsa_sparse_self_attn(q, k, v, m["col_idx"], m["col_cnt"], w.blk, want_lse=True)
        _status_ok(ws)
        return s, m, o, lse

    static = [t.clone() for t in inputs(0)]
    qa, kc, vc, q, k, v = static
    s0, m0, o0, lse0 = eager(*static)                       # also the warm-up that loads every kernel
    # caller-owned buffers of the captured step
    s = torch.empty_like(s0)
    lse_a = torch.empty((w.B, w.H, w.n_audio), dtype=torch.float32, device="cuda")
    out = {key: torch.empty_like(m0[key]) for key in ("block_scores", "col_idx", "col_cnt", "prot_tok", "prot_blk")}
    o, lse = torch.empty_like(o0), torch.empty_like(lse0)
    ws_c = torch.empty(av.avsa_cross_attn_scores_workspace_bytes(w.B, w.H, w.n_audio, w.n_video, w.d), dtype=torch.uint8, device="cuda")
    ws_m = torch.empty(av.avsa_build_block_mask_workspace_bytes(w.B, w.H, w.n_video, w.d, w.blk), dtype=torch.uint8, device="cuda")
    ws_a = torch.empty(av.avsa_sparse_self_attn_workspace_bytes(w.B, w.H, w.n_video, w.d, w.blk), dtype=torch.uint8, device="cuda")
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.graph(graph):
        av.avsa_cross_attn_scores(qa, kc, vc, scores=s, score_gamma=gamma, want_o=False, lse=lse_a, ws=ws_c)
        av.avsa_build_block_mask(q, k, s, n_protect, k_keep, w.blk, out=out, ws=ws_m)
        av.avsa_sparse_self_attn(q, k, v, out["col_idx"], out["col_cnt"], w.blk, o=o, lse=lse, ws=ws_a)
    for seed in (0, 5, 0):
        fresh = inputs(seed)
        for dst, src in zip(static, fresh):
            dst.copy_(src)
        for t in (s, o, lse, out["col_idx"], out["col_cnt"]):
            t.fill_(0)
        graph.replay()
        torch.cuda.synchronize()
        for ws_x in (ws_c, ws_m, ws_a):
            _status_ok(ws_x)
        assert av.avsa_redo_count(ws_a) == 0
        want_s, want_m, want_o, want_lse = eager(*fresh)
        assert torch.equal(s, want_s), f"seed {seed}: scores differ between replay and eager call"
        for key in ("col_idx", "col_cnt", "prot_tok", "prot_blk", "block_scores"):
            assert torch.equal(out[key], want_m[key]), f"seed {seed}: {key} differs between replay and eager call"
        assert torch.equal(o.view(torch.int16), want_o.view(torch.int16)), f"seed {seed}: O differs"
        assert torch.equal(lse, want_lse), f"seed {seed}: LSE differs"
    # the eager results of the last seed against the oracle
    idx, cnt = out["col_idx"].cpu().numpy(), out["col_cnt"].cpu().numpy()
    want, want_l = orc.masked_attention(_np64(q), _np64(k), _np64(v), idx, cnt, w.blk)
    _close(_np64(o), want, "graph replay O")
    _close_lse(_np64(lse), want_l, "graph replay lse")


# ------------------------------------------------------------------------------------------- token-exact protection
@pytest.mark.parametrize("name", ["tiny", "small128", "medium128"])
def test_token_exact_protection_matches_oracle(name):
    w = wl.WORKLOADS[name]
    q, k, v = wl.make_self_qkv(w, 6)
    _, _, _, s64 = _oracle_scores(w, 6)
    n_protect = orc.ceil_pct(w.protect_pct, w.n_video)
    k_keep = max(1, orc.ceil_pct(w.keep_pct, w.n_blocks))
    bs32 = orc.block_scores(_np64(q), _np64(k), w.blk).astype(np.float32)
    s32 = s64.astype(np.float32)
    idx, cnt, ptok, _ = orc.build_block_mask(bs32, s32, n_protect, k_keep, w.blk, w.n_video, protect_rows=False)
    m = av.avsa_build_block_mask(None, None, torch.from_numpy(s32).cuda(), n_protect, k_keep, w.blk,
                                 flags=av.AVSA_PROTECT_TOKENS | av.AVSA_USE_GIVEN_BLOCK_SCORES,
                                 block_scores=torch.from_numpy(bs32).cuda(), shape=(w.B, w.H, w.n_video, w.d))
    assert np.array_equal(m["col_idx"].cpu().numpy(), idx) and np.array_equal(m["col_cnt"].cpu().numpy(), cnt)
    assert np.array_equal(m["prot_tok"].cpu().numpy(), ptok)
    assert (cnt == k_keep).all()                                       # no block is made dense
    qc, kc, vc = q.cuda(), k.cuda(), v.cuda()
    o, lse, ws = av.avsa_sparse_self_attn(qc, kc, vc, m["col_idx"], m["col_cnt"], w.blk, want_lse=True)
    _status_ok(ws)
    ws2 = av.avsa_protected_rows_attn(qc, kc, vc, m["prot_tok"], n_protect, w.blk, o, lse=lse)
    _status_ok(ws2)
    want_o, want_l = orc.protected_attention_token_exact(_np64(q), _np64(k), _np64(v), idx, cnt, ptok, w.blk)
    _close(_np64(o), want_o, f"{name} token-exact O")
    _close_lse(_np64(lse), want_l, f"{name} token-exact lse")
    # a flag count that disagrees with n_protect is refused on the device and nothing is overwritten
    before = o.clone()
    ws3 = av.avsa_protected_rows_attn(qc, kc, vc, m["prot_tok"], n_protect + 1, w.blk, o)
    code, detail = av.avsa_read_status(ws3)
    assert code == av.AVSA_ERR_BAD_MASK and detail[2] == n_protect
    assert torch.equal(before, o)
    # zero protected tokens: a no-op
    av.avsa_protected_rows_attn(qc, kc, vc, torch.zeros_like(m["prot_tok"]), 0, w.blk, o)
    torch.cuda.synchronize()
    assert torch.equal(before, o)


# ------------------------------------------------------------------------------------------- Eq. 12-15
@pytest.mark.parametrize("Nv,Na,C", [(390, 40, 384), (2070, 72, 512), (5, 3, 8)])
def test_cache_indicators_match_oracle(Nv, Na, C):
    B = 2
    g = torch.Generator().manual_seed(Nv)
    y_v = torch.randn((B, Nv, C), generator=g).bfloat16()
    yhat_v = (y_v.float() + 0.2 * torch.randn((B, Nv, C), generator=g)).bfloat16()
    y_a = torch.randn((B, Na, C), generator=g).bfloat16()
    yhat_a = (y_a.float() + 0.05 * torch.randn((B, Na, C), generator=g)).bfloat16()
    prot = (torch.rand((B, Nv), generator=g) < 0.1).to(torch.uint8)
    prot[:, 0] = 1
    s_cur = torch.rand((B, Nv), generator=g)
    s_anchor = (s_cur + 0.3 * torch.rand((B, Nv), generator=g)).float()
    out, ws = av.avsa_cache_indicators(y_v.cuda(), yhat_v.cuda(), y_a.cuda(), yhat_a.cuda(), prot.cuda(), s_cur.cuda(),
                                       s_anchor.cuda())
    _status_ok(ws)
    got = out.cpu().numpy()
    for b in range(B):
        want = orc.cache_indicators(_np64(y_v[b]), _np64(yhat_v[b]), _np64(y_a[b]), _np64(yhat_a[b]), prot[b].numpy(),
                                    _np64(s_cur[b]), _np64(s_anchor[b]))
        for i, key in enumerate(("dv", "da", "dp", "ds", "dsync")):
            assert abs(got[b, i] - want[key]) <= 1e-4 * max(1.0, abs(want[key])), (b, key, got[b, i], want[key])
        assert bool(got[b, 5]) == want["reuse"]
    # no protected set and no saliency maps: those terms drop out
    out2, _ = av.avsa_cache_indicators(y_v.cuda(), y_v.cuda(), y_a.cuda(), y_a.cuda())
    assert np.allclose(out2.cpu().numpy()[:, :5], 0.0) and (out2.cpu().numpy()[:, 5] == 1.0).all()
    # reproducible bit for bit
    out3, _ = av.avsa_cache_indicators(y_v.cuda(), yhat_v.cuda(), y_a.cuda(), yhat_a.cuda(), prot.cuda(), s_cur.cuda(),
                                       s_anchor.cuda())
    assert torch.equal(out, out3)


@pytest.mark.parametrize("B,H,N,d,blk", [(1, 1, 1, 128, 128), (2, 1, 129, 128, 128), (3, 2, 65, 64, 64), (1, 5, 640, 128, 128)])
def test_degenerate_shapes_whole_path(B, H, N, d, blk):
    """One token, a one-token tail block, several batch items, one head: every call against the oracle."""
    NB = (N + blk - 1) // blk
    _whole_path_case(B, H, N, d, blk, 7, min(N, 3), max(1, NB // 2), B * 1000 + N)


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes_whole_path(seed):
    """Seeded random batch, heads, lengths (video and audio), tile size, protected count and kept count: every
    call of the path against the oracle, block-level and token-exact protection."""
    rng = np.random.default_rng(700 + seed)
    d = int(rng.choice([64, 128]))
    B, H = int(rng.integers(1, 3)), int(rng.integers(1, 5))
    N = int(rng.integers(2, 7 * d))
    NB = (N + d - 1) // d
    _whole_path_case(B, H, N, d, d, int(rng.integers(1, 300)), int(rng.integers(0, N // 4 + 2)),
                     int(rng.integers(1, NB + 1)), 800 + seed)


def _whole_path_case(B, H, N, d, blk, Na, n_protect, k_keep, seed):
    g = torch.Generator().manual_seed(seed)
    q, k, v = (torch.randn((B, H, N, d), generator=g).bfloat16() for _ in range(3))
    qa = torch.randn((B, H, Na, d), generator=g).bfloat16()
    gamma = 1.0 / (H * Na)
    o_a, lse_a, s, ws = av.avsa_cross_attn_scores(qa.cuda(), k.cuda(), v.cuda(), score_gamma=gamma)
    _status_ok(ws)
    want_oa, want_la, A = orc.cross_attention(_np64(qa), _np64(k), _np64(v))
    _close(_np64(o_a), want_oa, "cross O")
    _close_lse(_np64(lse_a), want_la, "cross lse")
    want_s = orc.column_scores(A, gamma=gamma)
    _close_scores(_np64(s), want_s, "scores")
    m = av.avsa_build_block_mask(q.cuda(), k.cuda(), s, n_protect, k_keep, blk)
    idx, cnt, ptok, pblk = orc.build_block_mask(m["block_scores"].cpu().numpy(), s.cpu().numpy(), n_protect, k_keep, blk, N)
    want_bs = orc.block_scores(_np64(q), _np64(k), blk)
    assert np.abs(m["block_scores"].cpu().numpy() - want_bs).max() <= 1e-4 * max(1.0, np.abs(want_bs).max())
    assert np.array_equal(m["col_idx"].cpu().numpy(), idx) and np.array_equal(m["col_cnt"].cpu().numpy(), cnt)
    assert np.array_equal(m["prot_tok"].cpu().numpy(), ptok) and np.array_equal(m["prot_blk"].cpu().numpy(), pblk)
    o, lse, ws3 = av.avsa_sparse_self_attn(q.cuda(), k.cuda(), v.cuda(), m["col_idx"], m["col_cnt"], blk, want_lse=True)
    _status_ok(ws3)
    want_o, want_l = orc.masked_attention(_np64(q), _np64(k), _np64(v), idx, cnt, blk)
    _close(_np64(o), want_o, "O")
    _close_lse(_np64(lse), want_l, "lse")
    # token-exact variant on the same inputs
    m2 = av.avsa_build_block_mask(q.cuda(), k.cuda(), s, n_protect, k_keep, blk, flags=av.AVSA_PROTECT_TOKENS)
    o2, lse2, _ = av.avsa_sparse_self_attn(q.cuda(), k.cuda(), v.cuda(), m2["col_idx"], m2["col_cnt"], blk, want_lse=True)
    ws4 = av.avsa_protected_rows_attn(q.cuda(), k.cuda(), v.cuda(), m2["prot_tok"], n_protect, blk, o2, lse=lse2)
    _status_ok(ws4)
    idx2, cnt2, ptok2, _ = orc.build_block_mask(m2["block_scores"].cpu().numpy(), s.cpu().numpy(), n_protect, k_keep, blk, N,
                                                protect_rows=False)
    want_o2, want_l2 = orc.protected_attention_token_exact(_np64(q), _np64(k), _np64(v), idx2, cnt2, ptok2, blk)
    _close(_np64(o2), want_o2, "token-exact O")
    _close_lse(_np64(lse2), want_l2, "token-exact lse")


def test_audio_branch_short_sequences():
    """The audio branch (m = a in Eq. 8-10) is the same three calls on a short sequence: fewer tokens than one
    block, and a two-block sequence with one protected block."""
    for (H, d, blk, N, k_keep, n_protect) in ((2, 64, 64, 40, 1, 4), (3, 128, 128, 256, 1, 13)):
        g = torch.Generator().manual_seed(N)
        q, k, v = (torch.randn((1, H, N, d), generator=g).bfloat16() for _ in range(3))
        s = torch.rand((1, N), generator=g)
        m = av.avsa_build_block_mask(q.cuda(), k.cuda(), s.cuda(), n_protect, k_keep, blk)
        idx, cnt, ptok, pblk = orc.build_block_mask(m["block_scores"].cpu().numpy(), s.numpy(), n_protect, k_keep, blk, N)
        assert np.array_equal(m["col_idx"].cpu().numpy(), idx) and np.array_equal(m["col_cnt"].cpu().numpy(), cnt)
        assert np.array_equal(m["prot_tok"].cpu().numpy(), ptok) and ptok.sum() == n_protect
        o, lse, ws = av.avsa_sparse_self_attn(q.cuda(), k.cuda(), v.cuda(), m["col_idx"], m["col_cnt"], blk, want_lse=True)
        _status_ok(ws)
        want_o, want_l = orc.masked_attention(_np64(q), _np64(k), _np64(v), idx, cnt, blk)
        _close(_np64(o), want_o, f"audio branch N={N} O")
        _close_lse(_np64(lse), want_l, f"audio branch N={N} lse")


def test_host_side_argument_errors():
    w = wl.WORKLOADS["tiny"]
    q, k, v = (t.cuda() for t in wl.make_self_qkv(w, 0))
    NB = w.n_blocks
    idx = torch.zeros((1, 2, NB, NB), dtype=torch.int32, device="cuda")
    cnt = torch.ones((1, 2, NB), dtype=torch.int32, device="cuda")
    with pytest.raises(av.AvsaError) as e:
        av.avsa_sparse_self_attn(q, k, v, idx, cnt, 32)
    assert e.value.status == av.AVSA_ERR_UNSUPPORTED
    with pytest.raises(av.AvsaError) as e:
        av.avsa_sparse_self_attn(q, k, v, idx, cnt, w.blk, ws=torch.empty(256, dtype=torch.uint8, device="cuda")[:8])
    assert e.value.status == av.AVSA_ERR_WORKSPACE
    with pytest.raises(av.AvsaError) as e:
        av.avsa_build_block_mask(q, k, None, 3, 1, w.blk)
    assert e.value.status == av.AVSA_ERR_INVALID_ARG
    with pytest.raises(av.AvsaError) as e:
        av.avsa_build_block_mask(q, k, None, 0, NB + 1, w.blk)
    assert e.value.status == av.AVSA_ERR_INVALID_ARG


# ------------------------------------------------------------------------------------------- caller-owned scratch
@pytest.mark.parametrize("name", ["tiny", "medium128"])
def test_results_do_not_depend_on_what_the_buffers_held_before(name):
    """Workspaces and outputs are caller-owned and arrive with arbitrary contents: every call must produce the
    same bits whether they were zero-filled or filled with 0xFF bytes (NaN patterns, negative counts)."""
    w = wl.WORKLOADS[name]
    qa, kc, vc = (t.cuda() for t in wl.make_cross_qkv(w, 3))
    q, k, v = (t.cuda() for t in wl.make_self_qkv(w, 3))
    n_protect = av.avsa_count_from_percent(w.protect_pct, w.n_video)
    k_keep = av.avsa_count_from_percent(w.keep_pct, w.n_blocks)
    NB = w.n_blocks
    C = w.H * w.d
    g = torch.Generator().manual_seed(9)
    y_v = torch.randn((w.B, w.n_video, C), generator=g).bfloat16().cuda()
    yhat_v = (y_v.float() * 1.1).bfloat16()
    y_a = torch.randn((w.B, w.n_audio, C), generator=g).bfloat16().cuda()
    yhat_a = (y_a.float() * 0.9).bfloat16()

    def run(fill):
        def buf(shape, dtype):
            t = torch.empty(shape, dtype=dtype, device="cuda")
            t.view(torch.uint8).fill_(fill)
            return t

        def scratch(nbytes):
            return buf((max(int(nbytes), 256),), torch.uint8)

        res = {}
        o_a, lse_a, s = buf(qa.shape, torch.bfloat16), buf(qa.shape[:3], torch.float32), buf((w.B, w.n_video), torch.float32)
        ws = scratch(av.avsa_cross_attn_scores_workspace_bytes(w.B, w.H, w.n_audio, w.n_video, w.d))
        av.avsa_cross_attn_scores(qa, kc, vc, scores=s, score_beta=0.0, score_gamma=1.0 / (w.H * w.n_audio), o=o_a,
                                  lse=lse_a, ws=ws)
        _status_ok(ws)
        res.update(o_a=o_a, lse_a=lse_a, s=s)
        for tag, flags in (("rows", av.AVSA_PROTECT_ROWS), ("tok", av.AVSA_PROTECT_TOKENS),
                           ("sum", av.AVSA_PROTECT_ROWS | av.AVSA_PROTECT_BLOCK_SUM)):
            out = dict(block_scores=buf((w.B, w.H, NB, NB), torch.float32), col_idx=buf((w.B, w.H, NB, NB), torch.int32),
                       col_cnt=buf((w.B, w.H, NB), torch.int32), prot_tok=buf((w.B, w.n_video), torch.uint8),
                       prot_blk=buf((w.B, NB), torch.uint8))
            ws = scratch(av.avsa_build_block_mask_workspace_bytes(w.B, w.H, w.n_video, w.d, w.blk))
            n = n_protect if tag != "sum" else max(1, NB // 4)
            av.avsa_build_block_mask(q, k, s, n, k_keep, w.blk, flags=flags, out=out, ws=ws)
            _status_ok(ws)
            for key, val in out.items():
                res[f"{tag}.{key}"] = val
        o, lse = buf(q.shape, torch.bfloat16), buf(q.shape[:3], torch.float32)
        ws = scratch(av.avsa_sparse_self_attn_workspace_bytes(w.B, w.H, w.n_video, w.d, w.blk))
        av.avsa_sparse_self_attn(q, k, v, res["tok.col_idx"], res["tok.col_cnt"], w.blk, o=o, lse=lse, ws=ws)
        _status_ok(ws)
        res.update(o_base=o.clone(), lse_base=lse.clone())
        ws = scratch(av.avsa_protected_rows_attn_workspace_bytes(w.B, w.H, w.n_video, w.d, w.blk, n_protect))
        av.avsa_protected_rows_attn(q, k, v, res["tok.prot_tok"], n_protect, w.blk, o, lse=lse, ws=ws)
        _status_ok(ws)
        res.update(o=o, lse=lse)
        ind = buf((w.B, 8), torch.float32)
        ws = scratch(av.avsa_cache_indicators_workspace_bytes(w.B, w.n_video, w.n_audio, C))
        av.avsa_cache_indicators(y_v, yhat_v, y_a, yhat_a, res["tok.prot_tok"], s, s, out=ind, ws=ws)
        _status_ok(ws)
        res["indicators"] = ind[:, :6].clone()
        torch.cuda.synchronize()
        return res

    a, b = run(0x00), run(0xFF)
    for key in a:
        assert torch.equal(a[key].view(torch.uint8), b[key].view(torch.uint8)), f"{key} depends on earlier buffer contents"


# ------------------------------------------------------------------------------------------- time-limited waits
def test_a_wait_that_nothing_ends_times_out_and_leaves_the_context_usable():
    """Every wait inside the tile kernels is time-limited.  The self-test kernel waits on a barrier that nothing
    signals: it must give up after the limit, report AVSA_ERR_TIMEOUT through the status record, and the next
    ordinary call on the same context must work."""
    ws = torch.empty(av.AVSA_STATUS_BYTES, dtype=torch.uint8, device="cuda")
    limit = 2_000_000                                           # about a millisecond
    av.avsa_selftest_bounded_wait(ws, limit)
    code, (where, item, waited_k) = av.avsa_read_status(ws)
    assert code == av.AVSA_ERR_TIMEOUT and where == 99 and item == 0
    assert limit // 1024 <= waited_k <= 4 * limit // 1024
    assert "timed out" in av.status_string(code)
    with pytest.raises(av.AvsaError):
        av.avsa_selftest_bounded_wait(ws, 3_000_000_000)        # limits beyond about a second are refused
    w = wl.WORKLOADS["tiny"]
    NB = w.n_blocks
    idx = np.broadcast_to(np.arange(NB, dtype=np.int32), (w.B, w.H, NB, NB)).copy()
    _run_sparse_case(w, 1, idx, np.full((w.B, w.H, NB), NB, np.int32))
