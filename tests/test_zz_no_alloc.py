"""The allocation-free mask entry point gives the same results as the workspace-taking one.

Collected last on purpose (file name), so a run that stops at the first failure has already run every
other test.  Some users of the library cannot allocate device memory at the point where they need the
mask (their host application has frozen its memory budget, or owns all of it); for them
avsa_build_block_mask_static keeps its scratch in an array inside the library.  The test calls it through
the C ABI twice in a row, on different inputs, because the array is shared between calls and keeps the
previous call's contents: the second result must not depend on what the first call left behind.
"""
import numpy as np
import pytest
import torch

from paper_2608_15522_b200 import binding as av
from paper_2608_15522_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _outputs(w, dev):
    NB = w.n_blocks
    return dict(block_scores=torch.empty((w.B, w.H, NB, NB), dtype=torch.float32, device=dev),
                col_idx=torch.empty((w.B, w.H, NB, NB), dtype=torch.int32, device=dev),
                col_cnt=torch.empty((w.B, w.H, NB), dtype=torch.int32, device=dev),
                prot_tok=torch.empty((w.B, w.n_video), dtype=torch.uint8, device=dev),
                prot_blk=torch.empty((w.B, NB), dtype=torch.uint8, device=dev))


def _compare(name, seed):
    w = wl.WORKLOADS[name]
    dev = torch.device("cuda", 0)
    q, k, _ = (t.to(dev) for t in wl.make_self_qkv(w, seed))
    scores = wl.uniform_flat(seed, 7, 0, w.B * w.n_video, "cpu").view(w.B, w.n_video).to(dev)
    n_protect = av.avsa_count_from_percent(w.protect_pct, w.n_video)
    k_keep = max(1, av.avsa_count_from_percent(w.keep_pct, w.n_blocks))
    want = av.avsa_build_block_mask(q, k, scores, n_protect, k_keep, w.blk)
    got = _outputs(w, dev)
    for t in got.values():
        t.fill_(123)                               # poison: every element must be written by the call
    av.avsa_build_block_mask_static(q, k, scores, n_protect, k_keep, w.blk, got)
    torch.cuda.synchronize()
    for key in ("col_idx", "col_cnt", "prot_tok", "prot_blk"):
        assert torch.equal(got[key], want[key]), (name, key)
    a, b = got["block_scores"].cpu().numpy(), want["block_scores"].cpu().numpy()
    assert np.abs(a - b).max() <= 1e-4 * max(1.0, np.abs(b).max())


def test_static_scratch_entry_point_matches_workspace_entry_point_twice_in_a_row():
    _compare("medium128", 11)      # fills most of what a later, smaller call will reuse
    _compare("tiny", 12)           # different shape and block size on the same array
    _compare("medium128", 13)


def test_static_scratch_entry_point_refuses_shapes_beyond_its_array():
    dev = torch.device("cuda", 0)
    B, H, N, d, blk = 1, 64, 128 * 400, 128, 128       # pooled means alone need 2 * 13 MB
    assert av.avsa_build_block_mask_workspace_bytes(B, H, N, d, blk) > av.AVSA_STATIC_SCRATCH_BYTES
    fake = torch.empty((B, H, 8, d), dtype=torch.bfloat16, device=dev)
    lib = av.load_library()
    t4 = av._t4(fake)
    one = torch.empty(16, dtype=torch.int32, device=dev)
    st = lib.avsa_build_block_mask_static(B, H, N, d, blk, t4, t4, None, 0, 1, 1, 0.0, av._ptr(one), av._ptr(one),
                                          av._ptr(one), None, None, None)
    assert st == av.AVSA_ERR_WORKSPACE               # refused on the host: nothing was enqueued
    torch.cuda.synchronize()
