"""The synthetic generators: shapes, determinism and the duplication structure they promise.  CPU only."""
import numpy as np
import torch

from paper_2502_11494_b200 import workloads as W


def test_config_shapes_and_budgets():
    assert [(w.B, w.S, w.n_vis, w.d, w.n_pivot, w.n_keep) for w in W.CONFIGS] == [
        (1, 676, 576, 4096, 8, 64), (64, 676, 576, 4096, 8, 64), (8, 2980, 2880, 4096, 16, 320),
        (4, 4708, 4608, 3584, 32, 512), (256, 2980, 2880, 4096, 8, 320)]
    assert all(w.vis_offset == 40 and w.S_out == w.S - w.n_vis + w.n_keep for w in W.CONFIGS)
    assert (128, 64) not in W.sweep_cells() and len(W.sweep_cells()) == 8


def test_samples_are_seeded_and_independent():
    w = W.LLAVA15_B64.with_(d=256)
    k0, h0 = W.make_sample(w, 3)
    k1, h1 = W.make_sample(w, 3)
    k2, _ = W.make_sample(w, 4)
    assert torch.equal(k0, k1) and torch.equal(h0, h1) and not torch.equal(k0, k2)
    assert k0.dtype == torch.bfloat16 and k0.shape == (w.S, w.d) and not torch.equal(k0, h0)
    kb, hb = W.make_batch(w, samples=range(3, 5))
    assert torch.equal(kb[0], k0) and torch.equal(kb[1], k2)


def _cos(x):
    x = x.double()
    x = x / x.norm(dim=1, keepdim=True)
    return x @ x.T


def test_cluster_structure_and_outliers():
    w = W.LLAVA15_B1
    k, h = W.make_sample(w, 0)
    vis = k[w.vis_offset:w.vis_offset + w.n_vis]
    l1 = vis.double().abs().sum(1)
    top = torch.topk(l1, 5).values
    assert top[3] / top[4] > 6.0                       # exactly four x8 outliers stand out
    c = _cos(vis)
    near = (c > 0.97).sum(1) - 1                       # same-centre tokens have cosine ~ 1/(1 + 0.1^2)
    assert near.double().mean() > 5 and (c > 0.97).double().mean() < 0.05
    off = c[c < 0.5]
    assert abs(off.mean()) < 0.01 and 0.010 < off.std() < 0.025   # other pairs ~ N(0, 1/sqrt(d))
    # hidden shares labels and outlier positions with keys
    hl1 = h[w.vis_offset:w.vis_offset + w.n_vis].double().abs().sum(1)
    assert set(torch.topk(hl1, 4).indices.tolist()) == set(torch.topk(l1, 4).indices.tolist())


def test_crops_share_centres_and_video_drifts():
    w = W.LLAVA_NEXT_B8.with_(d=512)
    k, _ = W.make_sample(w, 0)
    vis = k[w.vis_offset:w.vis_offset + w.n_vis]
    c = _cos(vis)                                       # full 2880 x 2880
    cross = c[:576, 576:1152]
    frac_dup = ((cross > 0.9).sum(1) > 0).double().mean().item()
    assert 0.15 < frac_dup < 0.45                      # ~30 % of a crop's tokens have a twin in another crop
    v = W.VIDEO_B4.with_(d=256)
    k, _ = W.make_sample(v, 0)
    vis = k[v.vis_offset:v.vis_offset + v.n_vis].double().view(32, 144, 256)
    step = (vis[1:] - vis[:-1]).flatten(1)
    ok = step.abs().max(1).values < 1.0                # frames without an outlier row
    assert 0.04 < step[ok].std() < 0.06                # frame t = frame t-1 + N(0, 0.05)
    n0, n31 = vis[0].norm(dim=1).median(), vis[31].norm(dim=1).median()
    assert n31 > n0                                    # drift variance accumulates


def test_bits_view_roundtrip():
    t = torch.tensor([[1.0, -2.0, 0.15625]], dtype=torch.bfloat16)
    b = W.bits(t)
    assert b.dtype == np.uint16 and b.tolist() == [[0x3F80, 0xC000, 0x3E20]]
