"""CPU oracle for the protected sparse video-attention path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 numpy statement of what the path computes, written from the paper's equations.
Only tests, the smoke check and the benchmark's CPU-baseline leg may import it; the product never
does, and this file shares no code with the CUDA sources.  Inputs are bf16 values widened exactly to
float64 by the caller; all arithmetic here is float64.

What follows the paper and what is this build's reading of it:

* ``cross_attention``, ``column_scores``           -- Eq. 1 and Eq. 2 (audio queries, video keys).
* ``protected_tokens``                             -- Eq. 3 / Eq. 8 (TopK with ceil(rho N) entries).
* ``masked_attention``                             -- Eq. 5-7 and Eq. 10 (softmax over kept keys only).
* ``block_mean_pool``, ``block_scores``, ``topk_blocks`` -- the base sparse pattern S_m.  The paper
  leaves S_m to "a standard sparse-attention method"; the rule here (mean-pooled Q/K block scores,
  per-head top-k) is this build's choice.  PARITY UNPINNED against the paper's own system for this
  rule; the functions are pinned against brute force and closed forms only.
* ``protected_attention_token_exact``               -- Eq. 9 / Eq. 11 on tokens (dense rows for protected tokens).
* ``cache_indicators``                             -- Eq. 12-15 (relative L1 changes, saliency drift, their maximum).
* ``protected_blocks``, ``build_block_mask``       -- Eq. 9 lifted from tokens to blocks: a block is
  protected iff it holds at least one protected token (a superset of the token-level rule).

Tie rule everywhere a top-k is taken: larger value first, then smaller index; NaN counts as -inf;
-0.0 equals +0.0.
"""
from __future__ import annotations

import numpy as np


def ceil_pct(pct: int, n: int) -> int:
    """ceil(pct/100 * n) in integer arithmetic (Eq. 8's ceiling)."""
    return (int(pct) * int(n) + 99) // 100


def _scale(d: int, scale) -> float:
    return float(scale) if scale else 1.0 / np.sqrt(float(d))


# ------------------------------------------------------------------------------------------------
# Eq. 1: cross-attention map, and its output rows
# ------------------------------------------------------------------------------------------------
def cross_attention(q, k, v, scale=None):
    """Eq. 1.  q [B,H,Nq,d], k,v [B,H,Nk,d] float64.

    Returns (O [B,H,Nq,d], lse [B,H,Nq] natural log, A [B,H,Nq,Nk]) with A = softmax(q k^T * scale).
    """
    q = np.asarray(q, np.float64); k = np.asarray(k, np.float64); v = np.asarray(v, np.float64)
    s = np.matmul(q, np.swapaxes(k, -1, -2)) * _scale(q.shape[-1], scale)     # [B,H,Nq,Nk]
    m = s.max(axis=-1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(axis=-1, keepdims=True)
    a = e / l
    lse = (m + np.log(l))[..., 0]
    return np.matmul(a, v), lse, a


# ------------------------------------------------------------------------------------------------
# Eq. 2: column mass summed over queries and heads, then the scalar Norm / running blend
# ------------------------------------------------------------------------------------------------
def column_scores(a, s_prev=None, beta=0.0, gamma=1.0):
    """Eq. 2 for one layer.  a [B,H,Nq,Nk] -> s [B,Nk] = beta*s_prev + gamma * sum_h sum_j a[.,h,j,:].

    gamma = 1/(H*Nq*|L_c|) gives the L1 Norm (scores of one layer sum to 1); beta = 1 accumulates
    layers; beta = alpha, gamma = (1-alpha)/(H*Nq) gives the running blend of Eq. 4.
    """
    c = np.asarray(a, np.float64).sum(axis=(1, 2))
    if s_prev is None:
        return gamma * c
    return beta * np.asarray(s_prev, np.float64) + gamma * c


# ------------------------------------------------------------------------------------------------
# Eq. 3 / Eq. 8: protected token set
# ------------------------------------------------------------------------------------------------
def _rank_key(x):
    x = np.array(x, np.float64, copy=True)
    x[np.isnan(x)] = -np.inf
    x[x == 0.0] = 0.0            # -0.0 -> +0.0
    return x


def topk_indices(x, k):
    """Indices of the k first entries of 1-D ``x`` under (value larger, then index smaller)."""
    key = _rank_key(x)
    order = np.argsort(-key, kind="stable")
    return order[: int(k)]


def protected_tokens(s, n_protect):
    """Eq. 8.  s [B,N] -> uint8 flags [B,N] with exactly n_protect ones per batch item."""
    s = np.asarray(s)
    flags = np.zeros(s.shape, np.uint8)
    for b in range(s.shape[0]):
        flags[b, topk_indices(s[b], n_protect)] = 1
    return flags


def protected_blocks(prot_tok, blk, min_tokens=1):
    """A block is protected iff it holds at least ``min_tokens`` protected tokens; with the default 1 this
    is the block lift of Eq. 9 (any protected token).  -> uint8 [B,NB]."""
    prot_tok = np.asarray(prot_tok)
    B, N = prot_tok.shape
    nb = (N + blk - 1) // blk
    out = np.zeros((B, nb), np.uint8)
    for b in range(B):
        count = [0] * nb
        for i in range(N):
            if prot_tok[b, i]:
                count[i // blk] += 1
        for j in range(nb):
            out[b, j] = 1 if count[j] >= max(1, min_tokens) else 0
    return out


def protected_blocks_by_sum(s, blk, n_blocks):
    """Variant of the block lift (not in the paper): protect the ``n_blocks`` blocks with the largest summed
    response, ties to the lowest block index.  The sum of a block is taken in fp64 and rounded to fp32, and the
    ranking is decided on that fp32 value.  s [B,N] -> uint8 [B,NB]."""
    s = np.asarray(s, np.float64)
    B, N = s.shape
    nb = (N + blk - 1) // blk
    out = np.zeros((B, nb), np.uint8)
    for b in range(B):
        sums = np.zeros(nb, np.float64)
        for j in range(nb):
            acc = 0.0
            for i in range(j * blk, min((j + 1) * blk, N)):
                acc += s[b, i]
            sums[j] = acc
        out[b, topk_indices(sums.astype(np.float32), n_blocks)] = 1
    return out


# ------------------------------------------------------------------------------------------------
# base sparse pattern S_m (this build's rule; the paper leaves it open)
# ------------------------------------------------------------------------------------------------
def block_mean_pool(x, blk):
    """x [B,H,N,d] -> [B,H,NB,d]: mean over the valid tokens of each block of ``blk`` tokens."""
    x = np.asarray(x, np.float64)
    B, H, N, d = x.shape
    nb = (N + blk - 1) // blk
    out = np.zeros((B, H, nb, d), np.float64)
    for j in range(nb):
        lo, hi = j * blk, min((j + 1) * blk, N)
        out[:, :, j, :] = x[:, :, lo:hi, :].sum(axis=2) / float(hi - lo)
    return out


def block_scores(q, k, blk, scale=None):
    """Bs[b,h,qb,kb] = mean-pooled q block . mean-pooled k block * scale."""
    qm = block_mean_pool(q, blk)
    km = block_mean_pool(k, blk)
    return np.matmul(qm, np.swapaxes(km, -1, -2)) * _scale(np.asarray(q).shape[-1], scale)


def topk_blocks(bs, k_keep):
    """keep[b,h,qb,kb] uint8: the k_keep best key blocks of every (head, query block) row."""
    bs = np.asarray(bs)
    B, H, NQ, NK = bs.shape
    keep = np.zeros(bs.shape, np.uint8)
    for b in range(B):
        for h in range(H):
            for i in range(NQ):
                keep[b, h, i, topk_indices(bs[b, h, i], k_keep)] = 1
    return keep


# ------------------------------------------------------------------------------------------------
# Eq. 9: protected mask, as per-row ascending column lists
# ------------------------------------------------------------------------------------------------
def apply_protection(keep, prot_blk, protect_rows=True, protect_cols=False):
    """Eq. 9 on blocks: a protected query block keeps every key block.  ``protect_cols``
    (not in the paper; an opt-in superset) also makes protected key blocks visible to every row."""
    keep = np.array(keep, np.uint8, copy=True)
    prot_blk = np.asarray(prot_blk)
    B, H, NQ, NK = keep.shape
    for b in range(B):
        for i in range(NQ):
            if protect_rows and prot_blk[b, i]:
                keep[b, :, i, :] = 1
        for j in range(NK):
            if protect_cols and prot_blk[b, j]:
                keep[b, :, :, j] = 1
    return keep


def keep_to_lists(keep):
    """keep [B,H,NQ,NK] -> (col_idx int32 [B,H,NQ,NK] ascending, padded with -1; col_cnt int32)."""
    keep = np.asarray(keep)
    B, H, NQ, NK = keep.shape
    idx = np.full((B, H, NQ, NK), -1, np.int32)
    cnt = np.zeros((B, H, NQ), np.int32)
    for b in range(B):
        for h in range(H):
            for i in range(NQ):
                cols = [j for j in range(NK) if keep[b, h, i, j]]
                cnt[b, h, i] = len(cols)
                idx[b, h, i, : len(cols)] = cols
    return idx, cnt


def build_block_mask(bs, scores, n_protect, k_keep, blk, n_tokens, protect_rows=True, protect_cols=False,
                     min_tokens=1, block_sum=False):
    """Block scores + token scores -> (col_idx, col_cnt, prot_tok, prot_blk), the whole mask step."""
    bs = np.asarray(bs)
    B = bs.shape[0]
    if block_sum:
        # n_protect counts BLOCKS here; every token of a protected block is flagged
        if n_protect > 0:
            prot_blk = protected_blocks_by_sum(scores, blk, n_protect)
        else:
            prot_blk = np.zeros((B, (n_tokens + blk - 1) // blk), np.uint8)
        prot_tok = np.repeat(prot_blk, blk, axis=1)[:, :n_tokens].astype(np.uint8)
    else:
        if n_protect > 0:
            prot_tok = protected_tokens(scores, n_protect)
        else:
            prot_tok = np.zeros((B, n_tokens), np.uint8)
        prot_blk = protected_blocks(prot_tok, blk, min_tokens)
    keep = apply_protection(topk_blocks(bs, k_keep), prot_blk, protect_rows, protect_cols)
    idx, cnt = keep_to_lists(keep)
    return idx, cnt, prot_tok, prot_blk


# ------------------------------------------------------------------------------------------------
# Eq. 10: attention under the protected block mask
# ------------------------------------------------------------------------------------------------
def masked_attention_rows(q_rows, k, v, cols, blk, scale=None):
    """Eq. 10 for the query rows of ONE (batch, head, query block).

    q_rows [R,d]; k,v [N,d]; ``cols`` = that row block's kept key-block indices.  The softmax runs
    over the kept keys only (the -inf entries of Eq. 6 contribute exp(-inf) = 0).
    Returns (O [R,d], lse [R]).
    """
    q_rows = np.asarray(q_rows, np.float64); k = np.asarray(k, np.float64); v = np.asarray(v, np.float64)
    N = k.shape[0]
    key_ids = np.concatenate([np.arange(j * blk, min((j + 1) * blk, N)) for j in cols])
    s = (q_rows @ k[key_ids].T) * _scale(q_rows.shape[-1], scale)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(axis=1, keepdims=True)
    return (e / l) @ v[key_ids], (m + np.log(l))[:, 0]


def masked_attention(q, k, v, col_idx, col_cnt, blk, scale=None):
    """Eq. 10 for whole tensors.  q,k,v [B,H,N,d] -> (O [B,H,N,d], lse [B,H,N])."""
    q = np.asarray(q, np.float64)
    B, H, N, d = q.shape
    out = np.zeros((B, H, N, d), np.float64)
    lse = np.zeros((B, H, N), np.float64)
    nb = (N + blk - 1) // blk
    for b in range(B):
        for h in range(H):
            for i in range(nb):
                lo, hi = i * blk, min((i + 1) * blk, N)
                cols = [int(c) for c in col_idx[b, h, i, : int(col_cnt[b, h, i])]]
                out[b, h, lo:hi], lse[b, h, lo:hi] = masked_attention_rows(
                    q[b, h, lo:hi], k[b, h], v[b, h], cols, blk, scale)
    return out, lse


def protected_attention_token_exact(q, k, v, col_idx, col_cnt, prot_tok, blk, scale=None):
    """Eq. 11 read on tokens: rows of protected tokens are dense attention rows (Eq. 5), every other row
    follows the sparse pattern given by the lists (Eq. 7).  The lists hold the base pattern only.
    q,k,v [B,H,N,d]; prot_tok [B,N] -> (O [B,H,N,d], lse [B,H,N])."""
    q = np.asarray(q, np.float64); k = np.asarray(k, np.float64); v = np.asarray(v, np.float64)
    out, lse = masked_attention(q, k, v, col_idx, col_cnt, blk, scale)
    B, H, N, d = q.shape
    for b in range(B):
        rows = np.nonzero(np.asarray(prot_tok)[b])[0]
        if len(rows) == 0:
            continue
        for h in range(H):
            s = (q[b, h, rows] @ k[b, h].T) * _scale(d, scale)
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            l = e.sum(axis=1, keepdims=True)
            out[b, h, rows] = (e / l) @ v[b, h]
            lse[b, h, rows] = (m + np.log(l))[:, 0]
    return out, lse


def dense_attention(q, k, v, scale=None):
    """Eq. 5: softmax(q k^T * scale) v for [B,H,N,d] tensors."""
    o, lse, _ = cross_attention(q, k, v, scale)
    return o, lse


# ------------------------------------------------------------------------------------------------
# Eq. 12-15: synchronization-aware cache-reuse indicators
# ------------------------------------------------------------------------------------------------
def cache_indicators(y_v, yhat_v, y_a, yhat_a, prot_tok=None, s_cur=None, s_anchor=None, lambda_p=0.5, lambda_s=0.1,
                     tau=0.2, eps=1e-6):
    """One batch item.  y_v, yhat_v [Nv,C]; y_a, yhat_a [Na,C]; prot_tok [Nv] flags; s_cur, s_anchor [Nv].

    Returns dict(dv, da, dp, ds, dsync, reuse):  Eq. 12 relative L1 change of each stream, Eq. 13 the same over
    the protected video rows, Eq. 14 one minus the cosine of the saliency maps, Eq. 15 their weighted maximum
    and the reuse decision dsync < tau.
    """
    y_v = np.asarray(y_v, np.float64); yhat_v = np.asarray(yhat_v, np.float64)
    y_a = np.asarray(y_a, np.float64); yhat_a = np.asarray(yhat_a, np.float64)
    dv = np.abs(y_v - yhat_v).sum() / (np.abs(y_v).sum() + eps)
    da = np.abs(y_a - yhat_a).sum() / (np.abs(y_a).sum() + eps)
    dp = 0.0
    if prot_tok is not None:
        rows = np.nonzero(np.asarray(prot_tok))[0]
        dp = np.abs(y_v[rows] - yhat_v[rows]).sum() / (np.abs(y_v[rows]).sum() + eps)
    ds = 0.0
    if s_cur is not None and s_anchor is not None:
        a = np.asarray(s_cur, np.float64); c = np.asarray(s_anchor, np.float64)
        ds = 1.0 - float(a @ c) / (np.sqrt(float(a @ a)) * np.sqrt(float(c @ c)) + eps)
    dsync = max(dv, da, lambda_p * dp, lambda_s * ds)
    return dict(dv=dv, da=da, dp=dp, ds=ds, dsync=dsync, reuse=bool(dsync < tau))
