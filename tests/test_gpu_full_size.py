"""Parity at the full Ovi-class size, in the launch configuration the benchmark times.

The oracle cannot compute a whole layer in seconds, so: the mask is compared in full (bit-exact given the
same fp32 score tensors), the cross-attention on a sample of heads, and the sparse attention on sampled
query blocks (first, ragged last, protected and unprotected ones) at full key length -- rows of Eq. 10 are
independent, so any subset can be checked alone.
"""
import numpy as np
import pytest
import torch

from oracle import avsa_oracle as orc
from paper_2608_15522_b200 import binding as av
from paper_2608_15522_b200 import workloads as wl
from parity_bars import close_lse as _close_lse, close_o as _close, close_scores as _close_scores, np64 as _np64

pytestmark = pytest.mark.gpu

@pytest.fixture(scope="module")
def ovi():
    w = wl.WORKLOADS["ovi"]
    dev = torch.device("cuda", 0)
    q, k, v = wl.make_self_qkv(w, 0, dev)
    qa, kc, vc = wl.make_cross_qkv(w, 0, dev)
    return w, (q, k, v), (qa, kc, vc)


def test_ovi_cross_attention_sampled_heads(ovi):
    w, _, (qa, kc, vc) = ovi
    gamma = 1.0 / (w.H * w.n_audio)
    o, lse, s, ws = av.avsa_cross_attn_scores(qa, kc, vc, score_gamma=gamma)
    assert av.avsa_read_status(ws)[0] == av.AVSA_OK
    assert abs(float(s.sum()) - 1.0) < 2e-3
    for h in (0, 11, 23):
        want_o, want_lse, _ = orc.cross_attention(_np64(qa[:, h:h + 1]), _np64(kc[:, h:h + 1]), _np64(vc[:, h:h + 1]))
        _close(_np64(o[:, h:h + 1]), want_o, f"cross O head {h}")
        _close_lse(_np64(lse[:, h:h + 1]), want_lse, f"cross lse head {h}")
    # scores need every head: accumulate the oracle head by head (Eq. 2)
    want_s = np.zeros((w.B, w.n_video))
    for h in range(w.H):
        _, _, A = orc.cross_attention(_np64(qa[:, h:h + 1]), _np64(kc[:, h:h + 1]), _np64(vc[:, h:h + 1]))
        want_s = orc.column_scores(A, s_prev=want_s, beta=1.0, gamma=gamma)
    got_s = _np64(s)
    _close_scores(got_s, want_s, "ovi scores")
    # most of the response mass sits in the planted regions, and so does the protected set
    region = wl.region_mask(w, "cpu").numpy()
    n_protect = orc.ceil_pct(w.protect_pct, w.n_video)
    top = orc.topk_indices(want_s[0], n_protect)
    assert region[top].mean() > 0.9
    _protected_set_agrees(s, want_s, n_protect, w, "ovi")


# A token can change sides between the GPU's and the oracle's protected set only if its fp64 score lies within the
# element-wise score bar (5e-3 relative) of the selection threshold, on either side: twice that, 1e-2, is the margin.
SET_MARGIN = 1e-2


def _protected_set_agrees(s_gpu, s64, n_protect, w, what):
    """End to end (Eq. 3 / Eq. 8): the GPU's protected set, selected by the GPU from its own fp32 scores, against
    the oracle's, selected in fp64 from its own scores.  Tokens whose oracle score is clear of the threshold by
    more than the margin must agree; the rest (ties up to rounding) may fall either way; both sets have n_protect
    tokens per batch item."""
    bs = torch.zeros((w.B, w.H, w.n_blocks, w.n_blocks), dtype=torch.float32, device=s_gpu.device)
    m = av.avsa_build_block_mask(None, None, s_gpu, n_protect, 1, w.blk, flags=av.AVSA_PROTECT_ROWS |
                                 av.AVSA_USE_GIVEN_BLOCK_SCORES, block_scores=bs, shape=(w.B, w.H, w.n_video, w.d))
    got = m["prot_tok"].cpu().numpy().astype(bool)
    for b in range(w.B):
        want = orc.protected_tokens(s64[b:b + 1], n_protect)[0].astype(bool)
        assert got[b].sum() == want.sum() == n_protect
        thr = np.sort(s64[b])[::-1][n_protect - 1]
        clear_in = s64[b] > thr * (1.0 + SET_MARGIN)
        clear_out = s64[b] < thr * (1.0 - SET_MARGIN)
        overlap = (got[b] & want).sum() / float(n_protect)
        assert got[b][clear_in].all(), f"{what}: a token clearly above the threshold is missing (overlap {overlap:.4f})"
        assert not got[b][clear_out].any(), f"{what}: a token clearly below the threshold was protected (overlap {overlap:.4f})"
        assert overlap >= 0.98, f"{what}: protected sets overlap only {overlap:.4f}"


def test_ovi_reverse_direction_audio_saliency(ovi):
    """Video queries, audio keys at full size: audio-token saliency (column sums over 32760 video queries)."""
    w, _, (qa, kc, vc) = ovi
    q_video, k_audio, v_audio = kc, qa, qa
    gamma = 1.0 / (w.H * w.n_video)
    o, lse, s, ws = av.avsa_cross_attn_scores(q_video, k_audio, v_audio, score_gamma=gamma)
    assert av.avsa_read_status(ws)[0] == av.AVSA_OK
    want_s = np.zeros((w.B, w.n_audio))
    for h in range(w.H):
        want_o, want_lse, A = orc.cross_attention(_np64(q_video[:, h:h + 1]), _np64(k_audio[:, h:h + 1]),
                                                  _np64(v_audio[:, h:h + 1]))
        want_s = orc.column_scores(A, s_prev=want_s, beta=1.0, gamma=gamma)
        if h in (0, 23):
            _close(_np64(o[:, h:h + 1]), want_o, f"reverse O head {h}")
            _close_lse(_np64(lse[:, h:h + 1]), want_lse, f"reverse lse head {h}")
    got_s = _np64(s)
    assert abs(got_s.sum() - 1.0) < 2e-3
    _close_scores(got_s, want_s, "ovi reverse scores")


def test_ovi_mask_full_and_sparse_attention_sampled_blocks(ovi):
    w, (q, k, v), (qa, kc, vc) = ovi
    NB = w.n_blocks
    n_protect = av.avsa_count_from_percent(w.protect_pct, w.n_video)
    k_keep = av.avsa_count_from_percent(w.keep_pct, NB)
    assert (n_protect, k_keep, NB) == (1638, 64, 256)
    _, _, s, _ = av.avsa_cross_attn_scores(qa, kc, vc, score_gamma=1.0 / (w.H * w.n_audio))
    m = av.avsa_build_block_mask(q, k, s, n_protect, k_keep, w.blk)
    assert av.avsa_read_status(m["ws"])[0] == av.AVSA_OK
    # block scores against the oracle (fp32 vs fp64), head by head to bound memory
    bs_gpu = m["block_scores"].cpu().numpy()
    for h in (0, 7, 23):
        want = orc.block_scores(_np64(q[:, h:h + 1]), _np64(k[:, h:h + 1]), w.blk)
        assert np.abs(bs_gpu[:, h:h + 1] - want).max() <= 1e-4 * max(1.0, np.abs(want).max())
    # lists: the oracle selecting from the same fp32 tensors must agree bit for bit, everywhere
    idx, cnt, ptok, pblk = orc.build_block_mask(bs_gpu, s.cpu().numpy(), n_protect, k_keep, w.blk, w.n_video)
    assert np.array_equal(m["prot_tok"].cpu().numpy(), ptok)
    assert np.array_equal(m["prot_blk"].cpu().numpy(), pblk)
    assert np.array_equal(m["col_cnt"].cpu().numpy(), cnt)
    assert np.array_equal(m["col_idx"].cpu().numpy(), idx)
    assert ptok.sum() == n_protect and 0 < pblk.sum() < NB
    # executed fraction vs Eq. 16's kappa + rho and its block-lifted form
    pairs = cnt.sum() / float(w.H * NB * NB)
    p_b = pblk.mean()
    assert abs(pairs - (0.25 + p_b * 0.75)) < 1e-9 and pairs >= 0.25 + 0.05 - 1e-9
    # sparse attention on sampled query blocks at full key length
    o, lse, ws = av.avsa_sparse_self_attn(q, k, v, m["col_idx"], m["col_cnt"], w.blk, want_lse=True)
    assert av.avsa_read_status(ws)[0] == av.AVSA_OK
    # on this workload no row outgrows its first-tile reference: the timed launch is the fast kernel alone
    assert av.avsa_sparse_self_attn_redo_items(ws)[0] == 0
    # a second launch reproduces the first bit for bit (fixed accumulation order; a difference would be a race)
    # (the work queue hands the query tiles to different CTAs from run to run; every tile's arithmetic is fixed)
    o2 = torch.empty_like(o)
    lse2 = torch.empty_like(lse)
    for _ in range(8):
        av.avsa_sparse_self_attn(q, k, v, m["col_idx"], m["col_cnt"], w.blk, o=o2, lse=lse2, ws=ws)
        assert torch.equal(o, o2) and torch.equal(lse, lse2)
        o2.zero_()
    del o2, lse2
    rng = np.random.default_rng(0)
    prot = np.nonzero(pblk[0])[0]
    unprot = np.nonzero(pblk[0] == 0)[0]
    blocks = [0, NB - 1] + rng.choice(prot, 3, replace=False).tolist() + rng.choice(unprot, 3, replace=False).tolist()
    for h in (0, 13, 23):
        kh, vh = _np64(k[0, h]), _np64(v[0, h])
        for i in blocks:
            lo, hi = i * w.blk, min((i + 1) * w.blk, w.n_video)
            cols = [int(c) for c in idx[0, h, i, : cnt[0, h, i]]]
            want_o, want_l = orc.masked_attention_rows(_np64(q[0, h, lo:hi]), kh, vh, cols, w.blk)
            _close(_np64(o[0, h, lo:hi]), want_o, f"O head {h} block {i}")
            _close_lse(_np64(lse[0, h, lo:hi]), want_l, f"lse head {h} block {i}")


def _check_workload_sampled(w, seed, heads, n_blocks_each, token_exact=False, check_scores=False):
    """Whole path on a full-size workload; mask bit-exact everywhere, attention on sampled query blocks."""
    dev = torch.device("cuda", 0)
    q, k, v = wl.make_self_qkv(w, seed, dev)
    qa, kc, vc = wl.make_cross_qkv(w, seed, dev)
    NB = w.n_blocks
    n_protect = av.avsa_count_from_percent(w.protect_pct, w.n_video)
    k_keep = max(1, av.avsa_count_from_percent(w.keep_pct, NB))
    _, _, s, ws1 = av.avsa_cross_attn_scores(qa, kc, vc, score_gamma=1.0 / (w.H * w.n_audio))
    assert av.avsa_read_status(ws1)[0] == av.AVSA_OK
    assert abs(float(s.sum()) - w.B) < 2e-3 * w.B
    if check_scores:
        # Eq. 2 needs every head: raw column mass (gamma = 1) accumulated by the oracle head by head
        _, _, s_raw, _ = av.avsa_cross_attn_scores(qa, kc, vc, score_gamma=1.0, want_o=False)
        want_s = np.zeros((w.B, w.n_video))
        for h in range(w.H):
            _, _, A = orc.cross_attention(_np64(qa[:, h:h + 1]), _np64(kc[:, h:h + 1]), _np64(vc[:, h:h + 1]))
            want_s = orc.column_scores(A, s_prev=want_s, beta=1.0, gamma=1.0)
            del A
        _close_scores(_np64(s_raw), want_s, f"{w.name} scores (raw column mass)")
        _protected_set_agrees(s, want_s, n_protect, w, w.name)
    flags = av.AVSA_PROTECT_TOKENS if token_exact else av.AVSA_PROTECT_ROWS
    m = av.avsa_build_block_mask(q, k, s, n_protect, k_keep, w.blk, flags=flags)
    bs_gpu = m["block_scores"].cpu().numpy()
    idx, cnt, ptok, pblk = orc.build_block_mask(bs_gpu, s.cpu().numpy(), n_protect, k_keep, w.blk, w.n_video,
                                                protect_rows=not token_exact)
    assert np.array_equal(m["prot_tok"].cpu().numpy(), ptok)
    assert np.array_equal(m["prot_blk"].cpu().numpy(), pblk)
    assert np.array_equal(m["col_cnt"].cpu().numpy(), cnt)
    assert np.array_equal(m["col_idx"].cpu().numpy(), idx)
    o, lse, ws = av.avsa_sparse_self_attn(q, k, v, m["col_idx"], m["col_cnt"], w.blk, want_lse=True)
    assert av.avsa_read_status(ws)[0] == av.AVSA_OK
    if token_exact:
        ws2 = av.avsa_protected_rows_attn(q, k, v, m["prot_tok"], n_protect, w.blk, o, lse=lse)
        assert av.avsa_read_status(ws2)[0] == av.AVSA_OK
    rng = np.random.default_rng(seed)
    prot = np.nonzero(pblk[0])[0]
    unprot = np.nonzero(pblk[0] == 0)[0]
    blocks = [0, NB - 1]
    if len(prot):
        blocks += rng.choice(prot, min(n_blocks_each, len(prot)), replace=False).tolist()
    if len(unprot):
        blocks += rng.choice(unprot, min(n_blocks_each, len(unprot)), replace=False).tolist()
    for h in heads:
        qh, kh, vh = _np64(q[0, h]), _np64(k[0, h]), _np64(v[0, h])
        for i in blocks:
            lo, hi = i * w.blk, min((i + 1) * w.blk, w.n_video)
            cols = [int(c) for c in idx[0, h, i, : cnt[0, h, i]]]
            want_o, want_l = orc.masked_attention_rows(qh[lo:hi], kh, vh, cols, w.blk)
            if token_exact:                                   # Eq. 11: protected rows are dense rows
                rows = np.nonzero(ptok[0, lo:hi])[0]
                if len(rows):
                    d_o, d_l = orc.masked_attention_rows(qh[lo:hi][rows], kh, vh, list(range(NB)), w.blk)
                    want_o[rows], want_l[rows] = d_o, d_l
            _close(_np64(o[0, h, lo:hi]), want_o, f"{w.name} O head {h} block {i}")
            _close_lse(_np64(lse[0, h, lo:hi]), want_l, f"{w.name} lse head {h} block {i}")
    return pblk, cnt


@pytest.mark.parametrize("keep,protect", [(10, 0), (25, 5), (50, 20)])
def test_mid_sweep_points(keep, protect):
    w = wl.WORKLOADS["mid"].with_ratios(keep, protect)
    pblk, cnt = _check_workload_sampled(w, 1, heads=(0, 17), n_blocks_each=2)
    assert (w.n_video, w.n_blocks) == (17856, 140)
    if protect == 0:
        assert pblk.sum() == 0 and (cnt == av.avsa_count_from_percent(keep, 140)).all()


def test_mid_token_exact_protection():
    _check_workload_sampled(wl.WORKLOADS["mid"].with_ratios(25, 5), 2, heads=(5,), n_blocks_each=2, token_exact=True)


def test_ltx_class_long_sequence():
    w = wl.WORKLOADS["ltx"]
    assert (w.n_video, w.n_blocks, w.n_audio) == (49152, 384, 512)
    _check_workload_sampled(w, 0, heads=(0, 31), n_blocks_each=2, check_scores=True)


def test_ovi_token_exact_protection():
    """Eq. 9 / Eq. 11 on tokens at the size the benchmark quotes its token-exact time on."""
    _check_workload_sampled(wl.WORKLOADS["ovi"], 0, heads=(3, 20), n_blocks_each=2, token_exact=True)


def test_ltx_token_exact_protection():
    _check_workload_sampled(wl.WORKLOADS["ltx"], 0, heads=(9,), n_blocks_each=2, token_exact=True)
