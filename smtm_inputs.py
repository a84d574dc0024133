"""Seeded synthetic workloads for the SMTM semantic-memory hot path.

Only input generation lives here: class centroids, label sequences, feature-map
tensors, initial semantic centres.  None of the method's arithmetic (pooling,
similarity, exit rule, table or centre updates) is in this module; the CPU
oracle and the CUDA library are both fed from it and share nothing else.

The five named workloads have the shapes, label statistics (bounded Zipf long
tail, temporal repetition) and dtypes/layouts of CNN exit-layer activations on
video streams; they stand in for the paper's UCF101 / long-tail CIFAR-100
streams and trained backbones, which are not used.
"""
from __future__ import annotations

import functools
import math
from dataclasses import dataclass, field, replace
from typing import List, Optional, Tuple

import numpy as np
import torch

F32, F16, BF16 = 0, 1, 2
NCHW, NHWC = 0, 1
_TORCH_DTYPE = {F32: torch.float32, F16: torch.float16, BF16: torch.bfloat16}
ELEM_SIZE = {F32: 4, F16: 2, BF16: 2}


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: int
    layout: int
    B: int                                  # frames per step
    stages: Tuple[Tuple[int, int, int], ...]  # (C, H, W) per candidate exit layer
    n: int                                  # classes in global memory
    k_init: int
    k_min: int
    k_max: int
    S: int = 1                              # streams (independent fast memories)
    T: int = 1                              # steps
    tau: float = 0.8
    window_W: int = 16
    sigma: float = 0.5
    relu: bool = True
    zipf_s: Optional[float] = None          # None = uniform labels
    novel_frac: float = 0.0                 # share of frames from classes outside the memory
    n_novel: int = 0
    repeat_p: float = 0.0                   # per-stream probability of repeating the last label
    unit_centroids: bool = False            # centroids L2-normalised and used as centres (m = 1)
    warm_m: int = 32                        # update count attached to the initial centres
    forgetting: bool = False                # frequency table itself decays (the paper's rapidly-changing-scene setting)
    seed: int = 0

    @property
    def L(self) -> int:
        return len(self.stages)

    @property
    def dims(self) -> List[int]:
        return [s[0] for s in self.stages]

    def frame_bytes(self, layer: int) -> int:
        c, h, w = self.stages[layer]
        return c * h * w * ELEM_SIZE[self.dtype]

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


RESNET50 = ((256, 56, 56), (512, 28, 28), (1024, 14, 14), (2048, 7, 7))
MOBILENETV2 = ((24, 56, 56), (32, 28, 28), (96, 14, 14), (320, 7, 7))

C1 = Workload("c1_single_layer_fp32", F32, NCHW, 8, ((64, 56, 56),), n=10, k_init=10, k_min=10,
              k_max=10, sigma=0.3, relu=False, unit_centroids=True, warm_m=1)
C2 = Workload("c2_resnet50_bf16", BF16, NCHW, 64, RESNET50, n=100, k_init=10, k_min=10, k_max=10,
              sigma=0.5, zipf_s=1.1)
C3 = Workload("c3_mobilenetv2_fp16_nhwc", F16, NHWC, 256, MOBILENETV2, n=200, k_init=16, k_min=16,
              k_max=16, sigma=0.5, zipf_s=1.2, novel_frac=0.2, n_novel=50)
C4 = Workload("c4_large_cache_bf16", BF16, NCHW, 1024, ((2048, 7, 7),), n=1000, k_init=1000,
              k_min=1000, k_max=1000, sigma=1.0, zipf_s=1.0)
C5 = Workload("c5_streaming_bf16", BF16, NCHW, 512, (RESNET50[2], RESNET50[3]), n=500, k_init=8,
              k_min=8, k_max=64, S=512, T=64, sigma=0.5, zipf_s=1.1, repeat_p=0.85)
# VGG16 on 32x32 inputs (the paper's long-tail CIFAR-100 setting): 13 shallow exits with tiny
# maps, 100 classes, rapidly changing scenes, frequency table with forgetting.
VGG16_CIFAR = ((64, 32, 32), (64, 32, 32), (128, 16, 16), (128, 16, 16), (256, 8, 8), (256, 8, 8), (256, 8, 8),
               (512, 4, 4), (512, 4, 4), (512, 4, 4), (512, 2, 2), (512, 2, 2), (512, 2, 2))
C6 = Workload("c6_vgg16_cifar_fp16", F16, NCHW, 128, VGG16_CIFAR, n=100, k_init=5, k_min=5, k_max=20, S=128, T=8,
              window_W=4, sigma=0.5, zipf_s=1.0, repeat_p=0.2, forgetting=True)
WORKLOADS = {w.name: w for w in (C1, C2, C3, C4, C5, C6)}


def _rng(w: Workload, *salt: int) -> np.random.Generator:
    return np.random.default_rng([w.seed, *salt])


@functools.lru_cache(maxsize=8)
def centroids(w: Workload) -> List[np.ndarray]:
    """Per layer: float32 [n + n_novel][C_l], i.i.d. N(0,1), independent across layers."""
    out = []
    for l, d in enumerate(w.dims):
        mu = _rng(w, 1, l).standard_normal((w.n + w.n_novel, d))
        if w.unit_centroids:
            mu /= np.linalg.norm(mu, axis=1, keepdims=True)
        out.append(mu.astype(np.float32))
    return out


def zipf_pmf(n: int, s: float) -> np.ndarray:
    """Bounded Zipf: p(r) proportional to r^-s for rank r = 1..n; class id = r - 1."""
    p = np.arange(1, n + 1, dtype=np.float64) ** (-s)
    return p / p.sum()


def _draw_labels(w: Workload, rng: np.random.Generator, size: int) -> np.ndarray:
    if w.zipf_s is None:
        lab = rng.integers(0, w.n, size)
    else:
        lab = rng.choice(w.n, size=size, p=zipf_pmf(w.n, w.zipf_s))
    if w.novel_frac > 0:
        novel = rng.random(size) < w.novel_frac
        lab = np.where(novel, w.n + rng.integers(0, w.n_novel, size), lab)
    return lab.astype(np.int32)


def labels(w: Workload) -> np.ndarray:
    """int32 [T][B] centroid index of every frame (>= n means a class outside the memory).

    With S > 1 frame b of every step belongs to stream b (B == S); within a
    stream the previous label repeats with probability repeat_p."""
    rng = _rng(w, 2)
    out = np.empty((w.T, w.B), np.int32)
    out[0] = _draw_labels(w, rng, w.B)
    for t in range(1, w.T):
        fresh = _draw_labels(w, rng, w.B)
        keep = rng.random(w.B) < w.repeat_p
        out[t] = np.where(keep, out[t - 1], fresh)
    return out


def stream_ids(w: Workload) -> np.ndarray:
    if w.S == 1:
        return np.zeros(w.B, np.int32)
    assert w.B == w.S
    return np.arange(w.B, dtype=np.int32)


def fallback_labels(w: Workload, lab: np.ndarray) -> np.ndarray:
    """What the full network would answer: the true class, -1 for classes outside the memory."""
    return np.where(lab < w.n, lab, -1).astype(np.int32)


def _rectified_mean(mu: torch.Tensor, sigma: float) -> torch.Tensor:
    """E[max(mu + sigma z, 0)] for z ~ N(0,1): mu Phi(mu/sigma) + sigma phi(mu/sigma)."""
    t = mu / sigma
    cdf = 0.5 * (1.0 + torch.erf(t / math.sqrt(2.0)))
    pdf = torch.exp(-0.5 * t * t) / math.sqrt(2.0 * math.pi)
    return mu * cdf + sigma * pdf


def initial_centers(w: Workload) -> Tuple[List[np.ndarray], List[np.ndarray]]:
    """Per layer (float32 [n][C_l] centres, uint32 [n] update counts).

    unit_centroids: the centroids themselves, count 1.  Otherwise each centre is
    the expected per-channel activation of its class (closed form for the
    rectified Gaussian the frames are drawn from) plus the sampling noise a mean
    over warm_m training frames would carry, count warm_m."""
    cents, counts = [], []
    for l, (c, h, ww) in enumerate(w.stages):
        mu = torch.from_numpy(centroids(w)[l][: w.n]).double()
        if w.unit_centroids:
            sc = mu
        else:
            sc = _rectified_mean(mu, w.sigma) if w.relu else mu
            noise = torch.from_numpy(_rng(w, 3, l).standard_normal((w.n, c)))
            sc = sc + noise * (w.sigma / math.sqrt(w.warm_m * h * ww))
        cents.append(sc.float().numpy().copy())
        counts.append(np.full(w.n, w.warm_m, np.uint32))
    return cents, counts


def frames(w: Workload, layer: int, lab: np.ndarray, step: int = 0, device="cpu") -> torch.Tensor:
    """Feature maps of one step at one layer: centroid broadcast over H x W plus
    sigma N(0,1) noise, rectified when w.relu, cast to w.dtype, laid out per w.layout.
    Shape [B,C,H,W] (NCHW) or [B,H,W,C] (NHWC), contiguous."""
    c, h, ww = w.stages[layer]
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(((w.seed * 1_000_003 + step) * 64 + layer) * 2 + 1)
    mu = torch.from_numpy(centroids(w)[layer]).to(dev)[torch.from_numpy(lab.astype(np.int64)).to(dev)]
    B = lab.shape[0]
    if w.layout == NCHW:
        x = torch.randn((B, c, h, ww), generator=gen, device=dev, dtype=torch.float32)
        x.mul_(w.sigma).add_(mu[:, :, None, None])
    else:
        x = torch.randn((B, h, ww, c), generator=gen, device=dev, dtype=torch.float32)
        x.mul_(w.sigma).add_(mu[:, None, None, :])
    if w.relu:
        x.clamp_(min=0)
    return x.to(_TORCH_DTYPE[w.dtype]).contiguous()


def shape4(w: Workload, layer: int, B: Optional[int] = None) -> Tuple[int, int, int, int]:
    c, h, ww = w.stages[layer]
    return (w.B if B is None else B, c, h, ww)
