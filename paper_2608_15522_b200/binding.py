"""ctypes binding of libavsa.so: same names as the C ABI, argument marshalling only.

PyTorch appears here for device memory and the current stream; every step of the path runs in the
library's CUDA kernels.  There is no CPU fallback: without the built library, or on a machine
without a CUDA device, the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libavsa.so")

AVSA_OK = 0
AVSA_ERR_INVALID_ARG = 1
AVSA_ERR_UNSUPPORTED = 2
AVSA_ERR_WORKSPACE = 3
AVSA_ERR_CUDA = 4
AVSA_ERR_TIMEOUT = 5
AVSA_ERR_BAD_MASK = 6

AVSA_PROTECT_ROWS = 1
AVSA_PROTECT_COLS = 2
AVSA_USE_GIVEN_BLOCK_SCORES = 4
AVSA_PROTECT_TOKENS = 8
AVSA_PROTECT_BLOCK_SUM = 16


def AVSA_MIN_TOKENS_PER_BLOCK(n: int) -> int:
    """Flag bits: a block is protected only if it holds at least n protected tokens."""
    return (int(n) & 0xFF) << 8


EXPORTS = (
    "avsa_cross_attn_scores", "avsa_cross_attn_scores_workspace_bytes",
    "avsa_build_block_mask", "avsa_build_block_mask_workspace_bytes", "avsa_build_block_mask_static",
    "avsa_sparse_self_attn", "avsa_sparse_self_attn_workspace_bytes",
    "avsa_protected_rows_attn", "avsa_protected_rows_attn_workspace_bytes",
    "avsa_cache_indicators", "avsa_cache_indicators_workspace_bytes",
    "avsa_count_from_percent", "avsa_read_status", "avsa_selftest_bounded_wait", "avsa_status_string", "avsa_version",
)


class AvsaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class _Bf16Tensor4(ctypes.Structure):
    _fields_ = [("ptr", ctypes.c_void_p), ("stride_b", ctypes.c_int64), ("stride_h", ctypes.c_int64),
                ("stride_n", ctypes.c_int64)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads libavsa.so (built in-tree by ``build.py``) and declares the prototypes."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2608_15522_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    i, f, vp, sz, u = ctypes.c_int, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint
    T = _Bf16Tensor4
    lib.avsa_cross_attn_scores.argtypes = [i, i, i, i, i, T, T, T, vp, vp, vp, f, f, f, vp, sz, vp]
    lib.avsa_cross_attn_scores.restype = i
    lib.avsa_cross_attn_scores_workspace_bytes.argtypes = [i, i, i, i, i]
    lib.avsa_cross_attn_scores_workspace_bytes.restype = sz
    lib.avsa_build_block_mask.argtypes = [i, i, i, i, i, T, T, vp, i, i, u, f, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.avsa_build_block_mask.restype = i
    lib.avsa_build_block_mask_workspace_bytes.argtypes = [i, i, i, i, i]
    lib.avsa_build_block_mask_workspace_bytes.restype = sz
    lib.avsa_build_block_mask_static.argtypes = [i, i, i, i, i, T, T, vp, i, i, u, f, vp, vp, vp, vp, vp, vp]
    lib.avsa_build_block_mask_static.restype = i
    lib.avsa_sparse_self_attn.argtypes = [i, i, i, i, i, T, T, T, vp, vp, vp, vp, f, vp, sz, vp]
    lib.avsa_sparse_self_attn.restype = i
    lib.avsa_sparse_self_attn_workspace_bytes.argtypes = [i, i, i, i, i]
    lib.avsa_sparse_self_attn_workspace_bytes.restype = sz
    lib.avsa_protected_rows_attn.argtypes = [i, i, i, i, i, T, T, T, vp, i, vp, vp, f, vp, sz, vp]
    lib.avsa_protected_rows_attn.restype = i
    lib.avsa_protected_rows_attn_workspace_bytes.argtypes = [i, i, i, i, i, i]
    lib.avsa_protected_rows_attn_workspace_bytes.restype = sz
    lib.avsa_cache_indicators.argtypes = [i, i, i, i, vp, vp, vp, vp, vp, vp, vp, f, f, f, f, vp, vp, sz, vp]
    lib.avsa_cache_indicators.restype = i
    lib.avsa_cache_indicators_workspace_bytes.argtypes = [i, i, i, i]
    lib.avsa_cache_indicators_workspace_bytes.restype = sz
    lib.avsa_count_from_percent.argtypes = [i, i]
    lib.avsa_count_from_percent.restype = i
    lib.avsa_read_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int)]
    lib.avsa_read_status.restype = i
    lib.avsa_selftest_bounded_wait.argtypes = [vp, sz, ctypes.c_longlong, vp]
    lib.avsa_selftest_bounded_wait.restype = i
    lib.avsa_status_string.argtypes = [i]
    lib.avsa_status_string.restype = ctypes.c_char_p
    lib.avsa_version.argtypes = []
    lib.avsa_version.restype = i
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().avsa_status_string(int(status)).decode()


def avsa_version() -> int:
    return int(load_library().avsa_version())


def avsa_count_from_percent(pct: int, n: int) -> int:
    return int(load_library().avsa_count_from_percent(int(pct), int(n)))


# ------------------------------------------------------------------------------------------------
# marshalling helpers
# ------------------------------------------------------------------------------------------------
def _t4(x: torch.Tensor) -> _Bf16Tensor4:
    if x.dtype != torch.bfloat16 or x.dim() != 4 or not x.is_cuda:
        raise ValueError("expected a CUDA bf16 tensor [B,H,N,d]")
    if x.stride(3) != 1:
        raise ValueError("the head dimension must be contiguous")
    return _Bf16Tensor4(x.data_ptr(), x.stride(0), x.stride(1), x.stride(2))


def _null_t4() -> _Bf16Tensor4:
    return _Bf16Tensor4(None, 0, 0, 0)


def _ptr(x: Optional[torch.Tensor]):
    return None if x is None else ctypes.c_void_p(x.data_ptr())


def _stream(device) -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def _workspace(nbytes: int, device, ws: Optional[torch.Tensor]) -> torch.Tensor:
    if ws is not None:
        return ws          # the library checks its size
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def _check(status: int, where: str) -> None:
    if status != AVSA_OK:
        raise AvsaError(status, where)


AVSA_STATUS_BYTES = 256


def avsa_read_status(ws: torch.Tensor) -> Tuple[int, Tuple[int, int, int]]:
    """Synchronises the current stream and returns (status, (where, item, aux)) of a workspace."""
    detail = (ctypes.c_int * 3)()
    code = load_library().avsa_read_status(_ptr(ws), _stream(ws.device), detail)
    return int(code), (int(detail[0]), int(detail[1]), int(detail[2]))


# ------------------------------------------------------------------------------------------------
# the three calls
# ------------------------------------------------------------------------------------------------
def avsa_selftest_bounded_wait(ws: torch.Tensor, limit_cycles: int) -> None:
    """Enqueues the wait that nothing ends; read the outcome with avsa_read_status(ws)."""
    st = load_library().avsa_selftest_bounded_wait(_ptr(ws), ws.numel(), int(limit_cycles), _stream(ws.device))
    _check(st, "avsa_selftest_bounded_wait")


def avsa_cross_attn_scores_workspace_bytes(B, H, Nq, Nk, d) -> int:
    return int(load_library().avsa_cross_attn_scores_workspace_bytes(B, H, Nq, Nk, d))


def avsa_cross_attn_scores(q, k, v, scores=None, score_beta=0.0, score_gamma=1.0, softmax_scale=0.0,
                           want_o=True, want_scores=True, o=None, lse=None, ws=None):
    """Eq. 1-2.  q [B,H,Nq,d], k/v [B,H,Nk,d] bf16 CUDA.  Returns (o, lse, scores, ws)."""
    lib = load_library()
    B, H, Nq, d = q.shape
    Nk = k.shape[2]
    dev = q.device
    if want_o and o is None:
        o = torch.empty_strided(q.shape, q.stride(), dtype=torch.bfloat16, device=dev)
    if lse is None:
        lse = torch.empty((B, H, Nq), dtype=torch.float32, device=dev)
    if want_scores and scores is None:
        scores = torch.empty((B, Nk), dtype=torch.float32, device=dev)
        score_beta = 0.0
    ws = _workspace(avsa_cross_attn_scores_workspace_bytes(B, H, Nq, Nk, d), dev, ws)
    st = lib.avsa_cross_attn_scores(B, H, Nq, Nk, d, _t4(q), _t4(k), _t4(v), _ptr(o if want_o else None), _ptr(lse),
                                    _ptr(scores if want_scores else None), float(score_beta), float(score_gamma),
                                    float(softmax_scale), _ptr(ws), ws.numel(), _stream(dev))
    _check(st, "avsa_cross_attn_scores")
    return o, lse, scores, ws


def avsa_build_block_mask_workspace_bytes(B, H, N, d, blk) -> int:
    return int(load_library().avsa_build_block_mask_workspace_bytes(B, H, N, d, blk))


def avsa_build_block_mask(q, k, scores, n_protect, k_keep, blk, flags=AVSA_PROTECT_ROWS, softmax_scale=0.0,
                          block_scores=None, shape=None, out=None, ws=None):
    """Eq. 8-9 plus the block-score top-k.  Returns dict(block_scores, col_idx, col_cnt, prot_tok, prot_blk, ws).

    With AVSA_USE_GIVEN_BLOCK_SCORES pass ``block_scores`` [B,H,NB,NB] fp32 and ``shape`` = (B,H,N,d);
    q and k may then be None.
    """
    lib = load_library()
    if q is not None:
        B, H, N, d = q.shape
        dev = q.device
    else:
        B, H, N, d = shape
        dev = block_scores.device
    NB = (N + blk - 1) // blk
    out = out or {}
    if block_scores is None:
        block_scores = out.get("block_scores")
    if block_scores is None:
        block_scores = torch.empty((B, H, NB, NB), dtype=torch.float32, device=dev)
    col_idx = out.get("col_idx")
    if col_idx is None:
        col_idx = torch.empty((B, H, NB, NB), dtype=torch.int32, device=dev)
    col_cnt = out.get("col_cnt")
    if col_cnt is None:
        col_cnt = torch.empty((B, H, NB), dtype=torch.int32, device=dev)
    prot_tok = out.get("prot_tok")
    if prot_tok is None:
        prot_tok = torch.empty((B, N), dtype=torch.uint8, device=dev)
    prot_blk = out.get("prot_blk")
    if prot_blk is None:
        prot_blk = torch.empty((B, NB), dtype=torch.uint8, device=dev)
    ws = _workspace(avsa_build_block_mask_workspace_bytes(B, H, N, d, blk), dev, ws)
    st = lib.avsa_build_block_mask(B, H, N, d, blk, _t4(q) if q is not None else _null_t4(),
                                   _t4(k) if k is not None else _null_t4(), _ptr(scores), int(n_protect), int(k_keep),
                                   int(flags), float(softmax_scale), _ptr(block_scores), _ptr(col_idx), _ptr(col_cnt),
                                   _ptr(prot_tok), _ptr(prot_blk), _ptr(ws), ws.numel(), _stream(dev))
    _check(st, "avsa_build_block_mask")
    return dict(block_scores=block_scores, col_idx=col_idx, col_cnt=col_cnt, prot_tok=prot_tok, prot_blk=prot_blk, ws=ws)


AVSA_STATIC_SCRATCH_BYTES = 16 << 20


def avsa_build_block_mask_static(q, k, scores, n_protect, k_keep, blk, out, flags=AVSA_PROTECT_ROWS, softmax_scale=0.0):
    """avsa_build_block_mask without a workspace: the library's built-in scratch array is used.

    For callers that must not allocate.  Accordingly this wrapper allocates nothing either: every output
    tensor (block_scores, col_idx, col_cnt, and prot_tok / prot_blk if wanted) must be supplied in ``out``.  Shapes that
    need more scratch than AVSA_STATIC_SCRATCH_BYTES raise AvsaError(AVSA_ERR_WORKSPACE).  The first call
    on a device resolves the array's address; make it before any stream capture.  Calls share the array, so
    do not let two of them overlap on the GPU.
    """
    lib = load_library()
    B, H, N, d = q.shape
    st = lib.avsa_build_block_mask_static(B, H, N, d, blk, _t4(q), _t4(k), _ptr(scores), int(n_protect), int(k_keep),
                                          int(flags), float(softmax_scale), _ptr(out["block_scores"]),
                                          _ptr(out["col_idx"]), _ptr(out["col_cnt"]), _ptr(out.get("prot_tok")),
                                          _ptr(out.get("prot_blk")), _stream(q.device))
    _check(st, "avsa_build_block_mask_static")
    return out


def avsa_sparse_self_attn_workspace_bytes(B, H, N, d, blk) -> int:
    return int(load_library().avsa_sparse_self_attn_workspace_bytes(B, H, N, d, blk))


def avsa_sparse_self_attn(q, k, v, col_idx, col_cnt, blk, softmax_scale=0.0, want_lse=False, o=None, lse=None, ws=None):
    """Eq. 10.  Returns (o, lse or None, ws)."""
    lib = load_library()
    B, H, N, d = q.shape
    dev = q.device
    if o is None:
        o = torch.empty_strided(q.shape, q.stride(), dtype=torch.bfloat16, device=dev)
    if want_lse and lse is None:
        lse = torch.empty((B, H, N), dtype=torch.float32, device=dev)
    ws = _workspace(avsa_sparse_self_attn_workspace_bytes(B, H, N, d, blk), dev, ws)
    st = lib.avsa_sparse_self_attn(B, H, N, d, blk, _t4(q), _t4(k), _t4(v), _ptr(col_idx), _ptr(col_cnt), _ptr(o),
                                   _ptr(lse), float(softmax_scale), _ptr(ws), ws.numel(), _stream(dev))
    _check(st, "avsa_sparse_self_attn")
    return o, lse, ws


def avsa_redo_count(ws: torch.Tensor) -> int:
    """Diagnostic: number of work items that the last attention call on this workspace (sparse self-attention,
    cross-attention pass 1, protected rows) recomputed with the exact-rescaling kernel."""
    torch.cuda.synchronize(ws.device)
    return int(ws[16:20].view(torch.int32).item())


def avsa_sparse_self_attn_redo_items(ws: torch.Tensor):
    """Diagnostic: (count, int32 array) of the work items ((b*H + h)*NB + query block) that the last
    avsa_sparse_self_attn call on this workspace recomputed with the exact-rescaling kernel."""
    torch.cuda.synchronize(ws.device)
    n = int(ws[16:20].view(torch.int32).item())
    items = ws[AVSA_STATUS_BYTES:AVSA_STATUS_BYTES + 4 * n].view(torch.int32).cpu().numpy()
    return n, items


def avsa_protected_rows_attn_workspace_bytes(B, H, N, d, blk, n_protect) -> int:
    return int(load_library().avsa_protected_rows_attn_workspace_bytes(B, H, N, d, blk, n_protect))


def avsa_protected_rows_attn(q, k, v, prot_tok, n_protect, blk, o, lse=None, softmax_scale=0.0, ws=None):
    """Eq. 9 / Eq. 11 on tokens: overwrites the rows of the protected tokens in ``o`` (and ``lse``) with dense
    attention rows.  Returns ws."""
    lib = load_library()
    B, H, N, d = q.shape
    dev = q.device
    ws = _workspace(avsa_protected_rows_attn_workspace_bytes(B, H, N, d, blk, int(n_protect)), dev, ws)
    st = lib.avsa_protected_rows_attn(B, H, N, d, blk, _t4(q), _t4(k), _t4(v), _ptr(prot_tok), int(n_protect), _ptr(o),
                                      _ptr(lse), float(softmax_scale), _ptr(ws), ws.numel(), _stream(dev))
    _check(st, "avsa_protected_rows_attn")
    return ws


def avsa_cache_indicators_workspace_bytes(B, Nv, Na, C) -> int:
    return int(load_library().avsa_cache_indicators_workspace_bytes(B, Nv, Na, C))


def avsa_cache_indicators(y_v, yhat_v, y_a, yhat_a, prot_tok=None, s_cur=None, s_anchor=None, lambda_p=0.5,
                          lambda_s=0.1, tau=0.2, eps=1e-6, out=None, ws=None):
    """Eq. 12-15.  y_v/yhat_v bf16 [B,Nv,C], y_a/yhat_a bf16 [B,Na,C] (contiguous).  Returns (out [B,8], ws) with
    out[:, :6] = dv, da, dp, ds, dsync, reuse."""
    lib = load_library()
    B, Nv, C = y_v.shape
    Na = y_a.shape[1]
    dev = y_v.device
    for t in (y_v, yhat_v, y_a, yhat_a):
        if t.dtype != torch.bfloat16 or not t.is_contiguous() or not t.is_cuda:
            raise ValueError("expected contiguous CUDA bf16 tensors")
    if out is None:
        out = torch.empty((B, 8), dtype=torch.float32, device=dev)
    ws = _workspace(avsa_cache_indicators_workspace_bytes(B, Nv, Na, C), dev, ws)
    st = lib.avsa_cache_indicators(B, Nv, Na, C, _ptr(y_v), _ptr(yhat_v), _ptr(y_a), _ptr(yhat_a), _ptr(prot_tok),
                                   _ptr(s_cur), _ptr(s_anchor), float(lambda_p), float(lambda_s), float(tau),
                                   float(eps), _ptr(out), _ptr(ws), ws.numel(), _stream(dev))
    _check(st, "avsa_cache_indicators")
    return out, ws
