"""Seeded synthetic inputs for the Q-GenX hot path.

This module holds input generation only: no quantizer, codec or update arithmetic lives
here.  It serves both the CUDA library's tests/benchmark and the CPU oracle's tests; both
sides always receive byte-identical copies of the same generated buffer (a buffer made on
the GPU is copied to the host for the oracle, never regenerated).

Five workload recipes (shapes and distributions stand in for the paper's workloads:
dual vectors of min-max games / VI operators with additive oracle noise, and layer-wise,
heavy-tailed gradient-like tensors as in GAN training):

  c1  bilinear game  min_x max_y x^T A y, n=1024 (d=2048), A ~ N(0,1/n), z0 ~ N(0,1),
      K=4 workers, noise N(0, 0.1^2) per coordinate, bucket 512, 9 uniform levels.
  c2  K=8 vectors of d=2^24 i.i.d. N(0,1), bucket 8192, 17 adaptive levels.
  c3  16 tensors, sizes {1728, 36864, 73728, 147456, 294912, 589824, 1179648, 2359296}
      each twice, Student-t (nu=3) entries scaled per tensor by 10^U(-3,0), K=16,
      bucket 4096, 9 adaptive levels per tensor.
  c4  affine VI  V(x) = M x + b, M = (G - G^T)/2 + 0.1 I, G ~ N(0,1/n) n=8192, b ~ N(0,1),
      x0 = 0, K=8, noise N(0,1) per coordinate, bucket 4096, 17 adaptive levels.
  c5  K=32 noise vectors of d=2^26, mixture 0.9 N(0,1) + 0.1 N(0,100), diagonal operator
      D ~ U(0.01,1), x0 ~ N(0,1), bucket 16384, 17 adaptive levels.

Every generator takes `device` ("cpu" or "cuda") and returns torch tensors; a reduced size
can be requested so that the oracle finishes in seconds.
"""
from dataclasses import dataclass
from typing import List, Optional

import torch

C3_TENSOR_SIZES = [1728, 36864, 73728, 147456, 294912, 589824, 1179648, 2359296]


def _gen(seed: int, device: str) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def gaussian(shape, seed, device="cpu", std=1.0):
    g = _gen(seed, device)
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32) * std


def uniform(shape, seed, device="cpu", lo=0.0, hi=1.0):
    g = _gen(seed, device)
    return torch.rand(shape, generator=g, device=device, dtype=torch.float32) * (hi - lo) + lo


def gaussian_mixture_(out: torch.Tensor, seed, p_wide=0.1, std_wide=10.0, chunk=1 << 26):
    """Fill `out` in place with 0.9 N(0,1) + 0.1 N(0,100): a standard normal, scaled by 10 with
    probability 0.1.  Chunked so that very large buffers need only bounded temporaries."""
    dev = str(out.device)
    g = _gen(seed, dev)
    flat = out.view(-1)
    for lo in range(0, flat.numel(), chunk):
        part = flat[lo:lo + chunk]
        part.normal_(generator=g)
        pick = torch.rand(part.shape, generator=g, device=out.device, dtype=torch.float32) < p_wide
        part.mul_(1.0 + (std_wide - 1.0) * pick.to(torch.float32))
    return out


def gaussian_mixture(shape, seed, device="cpu", p_wide=0.1, std_wide=10.0):
    return gaussian_mixture_(torch.empty(shape, device=device, dtype=torch.float32), seed, p_wide, std_wide)


def student_t3(shape, seed, device="cpu"):
    """Student-t with 3 degrees of freedom: Z / sqrt(chi2_3 / 3)."""
    g = _gen(seed, device)
    z = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    chi = torch.zeros(shape, device=device, dtype=torch.float32)
    for _ in range(3):
        w = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
        chi += w * w
    return z / torch.sqrt(chi / 3.0)


@dataclass
class BilinearGame:          # c1
    A: torch.Tensor          # [n, n]
    z0: torch.Tensor         # [2n]
    noise: torch.Tensor      # [T, 2, K, 2n]  (iteration, {t, t+1/2}, worker, coordinate)
    K: int = 4
    bucket: int = 512
    nlev: int = 9
    seed: int = 1001


def c1_bilinear(n=1024, K=4, T=100, device="cpu", seed=1001, noise_std=0.1, bucket=512) -> BilinearGame:
    A = gaussian((n, n), seed, device, std=(1.0 / n) ** 0.5)
    z0 = gaussian((2 * n,), seed + 1, device)
    noise = gaussian((T, 2, K, 2 * n), seed + 2, device, std=noise_std)
    return BilinearGame(A, z0, noise, K=K, bucket=bucket, seed=seed)


@dataclass
class VectorBatch:           # c2
    v: torch.Tensor          # [K, d]
    bucket: int
    nlev: int
    seed: int


def c2_gaussian(K=8, d=1 << 24, device="cpu", seed=1002, bucket=8192, nlev=17) -> VectorBatch:
    return VectorBatch(gaussian((K, d), seed, device), bucket, nlev, seed)


@dataclass
class LayerwiseBatch:        # c3
    v: torch.Tensor          # [K, sum(sizes)]; tensors laid back to back
    sizes: List[int]
    scales: List[float]
    bucket: int = 4096
    nlev: int = 9
    seed: int = 1003


def c3_layerwise(K=16, sizes: Optional[List[int]] = None, device="cpu", seed=1003, bucket=4096) -> LayerwiseBatch:
    if sizes is None:
        sizes = [s for s in C3_TENSOR_SIZES for _ in range(2)]
    expo = uniform((len(sizes),), seed + 7, "cpu", lo=-3.0, hi=0.0)
    scales = [float(10.0 ** float(e)) for e in expo]
    parts = []
    for j, (n, sc) in enumerate(zip(sizes, scales)):
        parts.append(student_t3((K, n), seed + 100 + j, device) * sc)
    return LayerwiseBatch(torch.cat(parts, dim=1).contiguous(), list(sizes), scales, bucket=bucket, seed=seed)


@dataclass
class AffineVI:              # c4
    M: torch.Tensor          # [n, n] row-major
    b: torch.Tensor          # [n]
    x0: torch.Tensor         # [n]
    K: int = 8
    bucket: int = 4096
    nlev: int = 17
    seed: int = 1004
    noise_std: float = 1.0

    def noise(self, t: int, device=None):
        """Noise for iteration t (1-based): [2, K, n], drawn on demand from (seed, t)."""
        dev = str(self.M.device) if device is None else device
        return gaussian((2, self.K, self.M.shape[0]), self.seed * 100003 + t, dev, std=self.noise_std)


def c4_affine(n=8192, K=8, device="cpu", seed=1004, bucket=4096, noise_std=1.0) -> AffineVI:
    G = gaussian((n, n), seed, device, std=(1.0 / n) ** 0.5)
    M = (G - G.t()) * 0.5 + 0.1 * torch.eye(n, device=device, dtype=torch.float32)
    b = gaussian((n,), seed + 1, device)
    return AffineVI(M.contiguous(), b, torch.zeros(n, device=device), K=K, bucket=bucket, seed=seed,
                    noise_std=noise_std)


@dataclass
class DiagonalScale:         # c5
    D: torch.Tensor          # [d]
    x0: torch.Tensor         # [d]
    noise: torch.Tensor      # [2, K, d]: one noise set for V_t and one for V_{t+1/2}, reused every iteration
    K: int = 32
    bucket: int = 16384
    nlev: int = 17
    seed: int = 1005


def c5_diagonal(K=32, d=1 << 26, device="cpu", seed=1005, bucket=16384) -> DiagonalScale:
    D = uniform((d,), seed, device, lo=0.01, hi=1.0)
    x0 = gaussian((d,), seed + 1, device)
    noise = torch.empty((2, K, d), device=device, dtype=torch.float32)
    gaussian_mixture_(noise, seed + 2)
    return DiagonalScale(D, x0, noise, K=K, bucket=bucket, seed=seed)


def player_scales(shape, block: int, p: float, seed: int, device="cpu") -> torch.Tensor:
    """Random player updating / random block coordinate descent as a relative-noise oracle: the last axis is cut
    into blocks of `block` coordinates (players); every (leading index, block) is drawn independently with
    probability p and its coordinates get the scale 1/p, all others 0 -- so the scales have mean one."""
    d = shape[-1]
    nblk = (d + block - 1) // block
    g = torch.Generator(device="cpu").manual_seed(int(seed))
    drawn = (torch.rand(tuple(shape[:-1]) + (nblk,), generator=g) < p).to(torch.float32) / float(p)
    out = drawn.repeat_interleave(block, dim=-1)[..., :d].contiguous()
    return out.to(device)


def uniform_levels(nlev: int) -> torch.Tensor:
    """l_j = j/(nlev-1): the level table before the first fit."""
    return torch.arange(nlev, dtype=torch.float64).div(nlev - 1).to(torch.float32)
