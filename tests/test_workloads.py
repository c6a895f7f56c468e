"""The synthetic generators: shapes, determinism, chunk independence, planted structure."""
import numpy as np
import torch

from paper_2608_15522_b200 import workloads as wl
from oracle import avsa_oracle as orc


def test_shapes_and_counts_match_the_configs():
    w = wl.WORKLOADS
    assert (w["tiny"].n_video, w["tiny"].n_blocks) == (256, 4)
    assert (w["ovi"].n_video, w["ovi"].n_blocks) == (32760, 256)
    assert (w["mid"].n_video, w["mid"].n_blocks) == (17856, 140)
    assert (w["ltx"].n_video, w["ltx"].n_blocks) == (49152, 384)
    assert w["ovi"].n_video % 128 == 120 and w["mid"].n_video % 128 == 64
    assert int(wl.region_mask(w["tiny"], "cpu").sum()) == 32
    assert int(wl.region_mask(w["ovi"], "cpu").sum()) == 1600


def test_generator_is_deterministic_and_chunk_independent():
    a = wl.normal_flat(3, 1, 0, 1000, "cpu")
    b = torch.cat([wl.normal_flat(3, 1, 0, 400, "cpu"), wl.normal_flat(3, 1, 400, 600, "cpu")])
    assert torch.equal(a, b)
    assert not torch.equal(a, wl.normal_flat(4, 1, 0, 1000, "cpu"))
    assert not torch.equal(a, wl.normal_flat(3, 2, 0, 1000, "cpu"))
    x = wl.normal_flat(0, 0, 0, 200000, "cpu").double()
    assert abs(float(x.mean())) < 0.01 and abs(float(x.std()) - 1.0) < 0.01
    assert torch.isfinite(x).all()


def test_tiny_tensors_and_planted_region_attracts_audio_queries():
    w = wl.WORKLOADS["tiny"]
    q, k, v = wl.make_cross_qkv(w, 0)
    assert q.shape == (1, 2, 32, 64) and k.shape == (1, 2, 256, 64) and q.dtype == torch.bfloat16
    q2, k2, v2 = wl.make_cross_qkv(w, 0)
    assert torch.equal(q, q2) and torch.equal(k, k2) and torch.equal(v, v2)
    _, _, A = orc.cross_attention(q.double().numpy(), k.double().numpy(), v.double().numpy())
    s = orc.column_scores(A, gamma=1.0 / (w.H * w.n_audio))[0]
    reg = wl.region_mask(w, "cpu").numpy()
    assert s[reg].sum() > 0.6                                   # most cross-modal mass lands in the region
    top = orc.topk_indices(s, orc.ceil_pct(w.protect_pct, w.n_video))
    assert len(top) == 26 and reg[top].mean() > 0.9


def test_self_qkv_structure():
    w = wl.WORKLOADS["small128"]
    q, k, v = wl.make_self_qkv(w, 5)
    assert q.shape == (1, 3, 390, 128)
    assert abs(float(v.float().std()) - 1.0) < 0.05
    assert float(q.float().std()) > 1.2                          # N(0,1) plus a unit-power field
    assert not torch.equal(q, k)
