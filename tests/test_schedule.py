"""Lagged saliency reuse: Eq. 4's recurrence, the K-step update schedule and the one-step lag.

CPU part: the schedule driven by the oracle as back end, against a hand-written loop.
GPU part: the same loop through the library on the tiny workload, every step checked against the oracle.
"""
import numpy as np
import pytest
import torch

from oracle import avsa_oracle as orc
from paper_2608_15522_b200 import schedule as sch
from paper_2608_15522_b200 import workloads as wl


def _oracle_cross(q, k, v, scores=None, score_beta=0.0, score_gamma=1.0, want_scores=True, **_):
    o, lse, A = orc.cross_attention(q, k, v)
    if not want_scores:
        return o, lse, None, None
    return o, lse, orc.column_scores(A, s_prev=scores, beta=score_beta, gamma=score_gamma), None


def test_schedule_recurrence_and_lag_on_cpu():
    rng = np.random.default_rng(0)
    alpha, K, T = 0.3, 2, 7
    lag = sch.LaggedSaliency(alpha=alpha, update_every=K, cross_fn=_oracle_cross)
    s_hand, seen_by_mask = None, []
    for t in range(T):
        q, k, v = rng.standard_normal((1, 2, 3, 4)), rng.standard_normal((1, 2, 9, 4)), rng.standard_normal((1, 2, 9, 4))
        used = lag.scores_for_mask()
        seen_by_mask.append(None if used is None else used.copy())
        if s_hand is None:
            assert used is None                                   # nothing to protect from before the first update
        else:
            np.testing.assert_allclose(used, s_hand, rtol=1e-14)  # the mask of step t sees the cache of step t-1
        lag.after_cross_attention(t, q, k, v, norm_gamma=1.0 / 6)
        if t % K == 0:                                            # Eq. 4, by hand
            _, _, A = orc.cross_attention(q, k, v)
            s_t = A.sum(axis=(1, 2)) / 6
            s_hand = s_t if s_hand is None else alpha * s_hand + (1 - alpha) * s_t
    assert lag.updates == 4 and [lag.is_update_step(t) for t in range(4)] == [True, False, True, False]
    np.testing.assert_allclose(lag.s_bar, s_hand, rtol=1e-14)
    np.testing.assert_allclose(lag.s_bar.sum(), 1.0, rtol=1e-12)  # a blend of L1-normalised maps stays normalised
    with pytest.raises(ValueError):
        sch.LaggedSaliency(alpha=1.0)


@pytest.mark.gpu
def test_lagged_loop_tiny_matches_oracle_every_step():
    from paper_2608_15522_b200 import binding as av
    w = wl.WORKLOADS["tiny"]
    gamma = 1.0 / (w.H * w.n_audio)
    n_protect = av.avsa_count_from_percent(w.protect_pct, w.n_video)
    k_keep = av.avsa_count_from_percent(w.keep_pct, w.n_blocks)
    gpu = sch.LaggedSaliency(alpha=0.5, update_every=2)
    ref = sch.LaggedSaliency(alpha=0.5, update_every=2, cross_fn=_oracle_cross)
    f64 = lambda t: t.double().cpu().numpy()
    for step in range(5):
        seed = wl.loop_seed(step, 0)
        q, k, v = wl.make_self_qkv(w, seed)
        qa, kc, vc = wl.make_cross_qkv(w, seed)
        # video self-attention of this step: protected from the cache of the previous step
        s_gpu, s_ref = gpu.scores_for_mask(), ref.scores_for_mask()
        n_p = n_protect if s_gpu is not None else 0
        m = av.avsa_build_block_mask(q.cuda(), k.cuda(), s_gpu, n_p, k_keep, w.blk)
        o, _, ws = av.avsa_sparse_self_attn(q.cuda(), k.cuda(), v.cuda(), m["col_idx"], m["col_cnt"], w.blk)
        assert av.avsa_read_status(ws)[0] == av.AVSA_OK
        if s_ref is not None:
            from parity_bars import close_scores
            close_scores(f64(s_gpu), s_ref, f"blended saliency at step {step}")
        # the oracle selecting from the very fp32 tensors the GPU used must give the same lists
        scores32 = None if s_gpu is None else s_gpu.cpu().numpy()
        idx, cnt, ptok, _ = orc.build_block_mask(m["block_scores"].cpu().numpy(), scores32, n_p, k_keep, w.blk, w.n_video)
        assert np.array_equal(m["col_idx"].cpu().numpy(), idx) and np.array_equal(m["col_cnt"].cpu().numpy(), cnt)
        assert np.array_equal(m["prot_tok"].cpu().numpy(), ptok)
        want, _ = orc.masked_attention(f64(q), f64(k), f64(v), idx, cnt, w.blk)
        err = np.abs(f64(o) - want)
        assert (err / np.maximum(1.0, np.abs(want))).max() <= 1e-2
        assert np.linalg.norm(err) / np.linalg.norm(want) <= 5e-3
        # then the cross-attention of this step updates the caches (every second step here)
        gpu.after_cross_attention(step, qa.cuda(), kc.cuda(), vc.cuda(), norm_gamma=gamma)
        ref.after_cross_attention(step, f64(qa), f64(kc), f64(vc), norm_gamma=gamma)
    assert gpu.updates == ref.updates == 3
