"""Lagged saliency reuse (Sec. 4.1): the saliency cache of Eq. 4 and its update schedule.

In a dual-stream block the video self-attention runs before the audio-video cross-attention, so the
cross-attention map of step t cannot guide the self-attention of step t.  The method keeps a cached
saliency map, blends a fresh one into it every K steps (Eq. 4), and protects at step t from the cache as
it stood after step t-1 (Eq. 8).  This module only sequences calls of the library and owns the cache
tensor; all arithmetic runs in ``avsa_cross_attn_scores`` (the blend is its ``score_beta/score_gamma``).

alpha is not given in the paper (0.5 here is this build's choice); the paper updates every K = 4 steps.
"""
from __future__ import annotations

from typing import Callable, Optional


class LaggedSaliency:
    """Owns s_bar and decides, per denoising step, whether the column-score pass runs.

    ``cross_fn(q, k, v, scores, score_beta, score_gamma, want_scores)`` must behave like
    ``binding.avsa_cross_attn_scores`` and return ``(o, lse, scores, ws)``; it is injectable so that the
    schedule can be exercised without a GPU.
    """

    def __init__(self, alpha: float = 0.5, update_every: int = 4, cross_fn: Optional[Callable] = None):
        if not (0.0 <= alpha < 1.0) or update_every < 1:
            raise ValueError("need 0 <= alpha < 1 and update_every >= 1")
        self.alpha = float(alpha)
        self.update_every = int(update_every)
        self._cross_fn = cross_fn
        self.s_bar = None          # cache after the last finished step; None until the first update
        self.updates = 0

    def is_update_step(self, t: int) -> bool:
        return t % self.update_every == 0

    def scores_for_mask(self):
        """The saliency the mask of the *current* step may use: the cache as of the previous step (lag)."""
        return self.s_bar

    def after_cross_attention(self, t: int, q_audio, k_video, v_video, norm_gamma: float, **kwargs):
        """Runs the cross-attention of step t; on update steps also its score pass, blended into the cache:
        first update s_bar = s_t, later ones s_bar = alpha*s_bar + (1-alpha)*s_t (Eq. 4).  Returns (o, lse)."""
        cross = self._cross_fn
        if cross is None:
            from . import binding
            cross = binding.avsa_cross_attn_scores
        if not self.is_update_step(t):
            o, lse, _, _ = cross(q_audio, k_video, v_video, want_scores=False, **kwargs)
            return o, lse
        if self.s_bar is None:
            o, lse, s, _ = cross(q_audio, k_video, v_video, scores=None, score_beta=0.0, score_gamma=norm_gamma, **kwargs)
            self.s_bar = s
        else:
            o, lse, s, _ = cross(q_audio, k_video, v_video, scores=self.s_bar, score_beta=self.alpha,
                                 score_gamma=(1.0 - self.alpha) * norm_gamma, **kwargs)
            self.s_bar = s         # the library blends in place and hands the same buffer back
        self.updates += 1
        return o, lse
