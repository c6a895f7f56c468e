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


def _compare(name, seed, flags=av.AVSA_PROTECT_ROWS, with_flag_outputs=True, n_protect=None):
    w = wl.WORKLOADS[name]
    dev = torch.device("cuda", 0)
    q, k, _ = (t.to(dev) for t in wl.make_self_qkv(w, seed))
    scores = wl.uniform_flat(seed, 7, 0, w.B * w.n_video, "cpu").view(w.B, w.n_video).to(dev)
    if n_protect is None:
        n_protect = av.avsa_count_from_percent(w.protect_pct, w.n_video)
    k_keep = max(1, av.avsa_count_from_percent(w.keep_pct, w.n_blocks))
    want = av.avsa_build_block_mask(q, k, scores, n_protect, k_keep, w.blk, flags=flags)
    got = _outputs(w, dev)
    if not with_flag_outputs:                      # the flags then live in the library's array, the part of it
        del got["prot_tok"], got["prot_blk"]       # most exposed to what the previous call left there
    for t in got.values():
        t.fill_(123)                               # poison: every element must be written by the call
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info(dev)[0]
    av.avsa_build_block_mask_static(q, k, scores, n_protect, k_keep, w.blk, got, flags=flags)
    torch.cuda.synchronize()
    # the call allocates nothing: the device's free memory is what it was (the first call of the process may
    # load the module's kernels lazily; every later call must leave the figure untouched)
    if _compare.calls > 0:
        assert torch.cuda.mem_get_info(dev)[0] == free_before, "the allocation-free entry point changed free memory"
    _compare.calls += 1
    # same kernels, same inputs, same launch shapes: every output is bit-identical, the fp32 block scores included
    for key in got:
        assert torch.equal(got[key], want[key]), (name, key)


_compare.calls = 0


def test_static_scratch_entry_point_matches_workspace_entry_point_twice_in_a_row():
    _compare("medium128", 11)      # fills most of what a later, smaller call will reuse
    _compare("tiny", 12)           # different shape and block size on the same array
    _compare("medium128", 13)


def test_static_scratch_entry_point_with_its_flag_buffers_inside_the_array():
    """prot_tok / prot_blk not requested: the library keeps them in the shared array, where the previous call of
    another shape has left its own pooled means and flags; and the block-sum variant, whose sums and scratch
    flags live there too."""
    _compare("medium128", 21)
    _compare("tiny", 22, with_flag_outputs=False)
    _compare("medium128", 23, with_flag_outputs=False)
    _compare("tiny", 24, flags=av.AVSA_PROTECT_ROWS | av.AVSA_PROTECT_BLOCK_SUM, n_protect=1)
    _compare("medium128", 25, flags=av.AVSA_PROTECT_ROWS | av.AVSA_PROTECT_BLOCK_SUM, n_protect=3, with_flag_outputs=False)


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
