"""Seeded synthetic inputs shaped like the paper's MLLM workloads.

This module only draws random numbers and rounds them to bf16.  It holds none of the
reduction step's arithmetic and is the one module that both the CUDA path's callers and the
oracle's callers use, so that the two sides read the same bits.

The paper measures on LLaVA-1.5 (576 vision tokens), LLaVA-NeXT (2880) and video models; its
datasets and weights are not available, so these generators imitate only the shapes and a
duplication structure: vision tokens are noisy copies of a few cluster centres (duplicates
exist), a few tokens have an outlying norm, text tokens surround the vision block.

Recipe (all draws in fp32, then one round-to-nearest-even cast to bf16):
  * ``N(mu, sigma)``: the second argument is the standard deviation.
  * keys: vision row = centre[label] + N(0, noise); hidden uses the same labels with
    independent centres and noise; text rows are iid N(0, 1).
  * 4 vision tokens per sample (uniform without replacement) are multiplied by 8 after all other
    steps, at the same indices in keys and hidden.
  * sample b of workload w uses seed 1_000_003 * w.seed_base + b on the chosen device's generator
    (CPU and CUDA generators give different streams; a test or bench generates once and hands
    the same bits to both sides).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional

import torch

N_OUTLIERS = 4
OUTLIER_SCALE = 8.0


@dataclass(frozen=True)
class Workload:
    name: str
    seed_base: int
    B: int
    n_before: int
    n_vis: int
    n_after: int
    d: int
    n_pivot: int
    n_keep: int
    kind: str  # "cluster" | "crops" | "video"
    centres_lo: int = 48
    centres_hi: int = 48  # inclusive; per-sample uniform in [lo, hi]
    noise: float = 0.1
    n_crops: int = 1
    shared_frac: float = 0.0
    n_frames: int = 1
    drift: float = 0.0

    @property
    def S(self) -> int:
        return self.n_before + self.n_vis + self.n_after

    @property
    def vis_offset(self) -> int:
        return self.n_before

    @property
    def S_out(self) -> int:
        return self.S - self.n_vis + self.n_keep

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five benchmark configurations (text block 40 before / 60 after in all of them).
LLAVA15_B1 = Workload("llava15_b1", 1, 1, 40, 576, 60, 4096, 8, 64, "cluster")
LLAVA15_B64 = Workload("llava15_b64", 2, 64, 40, 576, 60, 4096, 8, 64, "cluster", centres_lo=16, centres_hi=128)
LLAVA_NEXT_B8 = Workload("llava_next_b8", 3, 8, 40, 2880, 60, 4096, 16, 320, "crops", n_crops=5, shared_frac=0.3)
VIDEO_B4 = Workload("video_b4", 4, 4, 40, 4608, 60, 3584, 32, 512, "video", n_frames=32, drift=0.05)
SWEEP_B256 = Workload("sweep_b256", 5, 256, 40, 2880, 60, 4096, 8, 320, "crops", n_crops=5, shared_frac=0.3)

CONFIGS = (LLAVA15_B1, LLAVA15_B64, LLAVA_NEXT_B8, VIDEO_B4, SWEEP_B256)

# Two more shapes the paper applies the step to (appendix): a vision-language-action model that keeps 56 of its 256
# image tokens per control step (batch of 16 environments, an instruction of a few tokens after the image), and
# audio tokens of a long utterance reduced by 20 / 30 / 50 % with 8 pivots (1500 tokens of width 3072 stand for two
# minutes of speech; consecutive frames drift like the video generator's).  Not benchmark configurations: parity
# cases and `bench.py --workload` choices.
VLA_B16 = Workload("vla_b16", 6, 16, 1, 256, 20, 4096, 8, 56, "cluster", centres_lo=24, centres_hi=64)
AUDIO_B8 = Workload("audio_b8", 7, 8, 10, 1500, 30, 3072, 8, 750, "video", n_frames=100, drift=0.05)
AUDIO_KEEP = (1200, 1050, 750)  # 20 %, 30 %, 50 % of the audio tokens removed
EXTRA = (VLA_B16, AUDIO_B8)
SWEEP_PIVOTS = (8, 32, 128)
SWEEP_KEEP = (64, 320, 640)


def sweep_cells():
    """(n_pivot, n_keep) cells of the bandwidth sweep; cells with more pivots than kept tokens are invalid."""
    return [(p, k) for p in SWEEP_PIVOTS for k in SWEEP_KEEP if p <= k]


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _randn(shape, g, device, std: float = 1.0):
    x = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    return x if std == 1.0 else x * std


def _clustered(n_tok: int, d: int, centres_k, centres_h, noise: float, g, device):
    """n_tok tokens, each a uniformly chosen centre plus noise; same labels for keys and hidden."""
    C = centres_k.shape[0]
    labels = torch.randint(0, C, (n_tok,), generator=g, device=device)
    k = centres_k[labels] + _randn((n_tok, d), g, device, noise)
    h = centres_h[labels] + _randn((n_tok, d), g, device, noise)
    return k, h


def _vision_block(w: Workload, g, device):
    d = w.d
    if w.kind == "cluster":
        if w.centres_lo == w.centres_hi:
            C = w.centres_lo
        else:
            C = int(torch.randint(w.centres_lo, w.centres_hi + 1, (1,), generator=g, device=device).item())
        ck, ch = _randn((C, d), g, device), _randn((C, d), g, device)
        return _clustered(w.n_vis, d, ck, ch, w.noise, g, device)
    if w.kind == "crops":
        per = w.n_vis // w.n_crops
        C = w.centres_lo
        n_shared = int(w.shared_frac * C)  # centres that every crop of the sample has in common
        sk, sh = _randn((n_shared, d), g, device), _randn((n_shared, d), g, device)
        ks, hs = [], []
        for _ in range(w.n_crops):
            pk, ph = _randn((C - n_shared, d), g, device), _randn((C - n_shared, d), g, device)
            k, h = _clustered(per, d, torch.cat([sk, pk]), torch.cat([sh, ph]), w.noise, g, device)
            ks.append(k)
            hs.append(h)
        return torch.cat(ks), torch.cat(hs)
    if w.kind == "video":
        per = w.n_vis // w.n_frames
        C = w.centres_lo
        ck, ch = _randn((C, d), g, device), _randn((C, d), g, device)
        k, h = _clustered(per, d, ck, ch, w.noise, g, device)
        ks, hs = [k], [h]
        for _ in range(1, w.n_frames):  # frame t = frame t-1 + drift noise
            k = k + _randn((per, d), g, device, w.drift)
            h = h + _randn((per, d), g, device, w.drift)
            ks.append(k)
            hs.append(h)
        return torch.cat(ks), torch.cat(hs)
    raise ValueError("unknown workload kind %r" % w.kind)


def make_sample(w: Workload, b: int, device="cpu"):
    """One sample: (keys [S, d] bf16, hidden [S, d] bf16)."""
    g = _gen(device, 1_000_003 * w.seed_base + b)
    vk, vh = _vision_block(w, g, device)
    out = torch.randperm(w.n_vis, generator=g, device=device)[:N_OUTLIERS]
    vk[out] *= OUTLIER_SCALE
    vh[out] *= OUTLIER_SCALE
    parts_k, parts_h = [], []
    for n_txt in (w.n_before, None, w.n_after):
        if n_txt is None:
            parts_k.append(vk)
            parts_h.append(vh)
        else:
            parts_k.append(_randn((n_txt, w.d), g, device))
            parts_h.append(_randn((n_txt, w.d), g, device))
    keys = torch.cat(parts_k).to(torch.bfloat16)
    hidden = torch.cat(parts_h).to(torch.bfloat16)
    return keys, hidden


def make_batch(w: Workload, device="cpu", samples: Optional[range] = None, pin: bool = False):
    """(keys [B, S, d], hidden [B, S, d]) bf16 on ``device``; ``samples`` selects a sub-range of the batch."""
    idx = list(range(w.B)) if samples is None else list(samples)
    kw = {"pin_memory": True} if (pin and str(device) == "cpu") else {}
    keys = torch.empty((len(idx), w.S, w.d), dtype=torch.bfloat16, device=device, **kw)
    hidden = torch.empty_like(keys, **kw) if not kw else torch.empty((len(idx), w.S, w.d), dtype=torch.bfloat16, **kw)
    for i, b in enumerate(idx):
        k, h = make_sample(w, b, device)
        keys[i].copy_(k)
        hidden[i].copy_(h)
    return keys, hidden


def bits(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 array of its bit patterns (host copy)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")
