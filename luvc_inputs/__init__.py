"""Seeded synthetic inputs shaped like the paper's workloads.

This module is the one piece shared by the CPU oracle's tests and the CUDA
path's tests and benchmark.  It holds none of the method's arithmetic: it only
draws smooth random fields, noise, outliers and a projection matrix.

The paper evaluates on public image / video benchmark suites; none of their
items is used here.  What is kept is the shape of the work: ViT patch grids
(24x24 at D=1024, up to 128x128 at D=1280), per-frame video grids, and LLM
hidden states (D=3584 / 4096) over 64 to 16384 visual tokens.

Determinism: every random parameter (cosine amplitudes, frequencies, phases,
outlier positions, rectangles, drifts) comes from numpy's counter-based Philox
generator keyed by the seed, so it is the same on every machine.  Bulk iid
noise comes from a torch generator seeded with the same seed on the device the
tensor is built on (CPU and CUDA streams differ, each is reproducible).
"""
from __future__ import annotations

import math

import numpy as np
import torch

TWO_PI = 2.0 * math.pi

# (name, B, H, W, D_vit, target, D_llm, keeps, dtype) for the five configurations.
CONFIGS = {
    0: dict(name="single-image-fp32", B=1, H=24, W=24, D=1024, target=144, D_llm=4096, keep=(64,), dtype="f32"),
    1: dict(name="batch32-outliers", B=32, H=24, W=24, D=1024, target=64, D_llm=4096, keep=(32,), dtype="bf16"),
    2: dict(name="highres-72x72", B=8, H=72, W=72, D=1280, target=1296, D_llm=3584, keep=(324, 130, 65), dtype="bf16"),
    3: dict(name="video-16x36x36", B=32, H=36, W=36, D=1280, target=162, D_llm=3584, keep=(648,), dtype="bf16",
            frames=16, videos=2),
    4: dict(name="stress", B=4, H=128, W=128, D=1280, target=2048, D_llm=4096, keep=(1638, 4096, 8192),
            dtype="bf16", spu_B=8, spu_N=16384, cutoffs=(0.05, 0.125, 0.25)),
}


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=int(seed)))


def _noise(shape, std: float, seed: int, device) -> torch.Tensor:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) + 0x5EED)
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32) * std


def _t(a, device) -> torch.Tensor:
    return torch.as_tensor(np.asarray(a, dtype=np.float32), device=device)


def smooth_field_2d(H, W, D, seed, ncos=8, device="cpu", shift=(0.0, 0.0), params=None) -> torch.Tensor:
    """[H,W,D] float32: per channel a sum of `ncos` random 2D cosines, amplitude N(0,1),
    frequencies U(-2,2) cycles per image side, phase U[0, 2 pi); sampled at (h+shift_h, w+shift_w)."""
    if params is None:
        r = _rng(seed)
        params = dict(a=r.standard_normal((ncos, D)), u=r.uniform(-2, 2, (ncos, D)),
                      v=r.uniform(-2, 2, (ncos, D)), phi=r.uniform(0, TWO_PI, (ncos, D)))
    hh = (torch.arange(H, device=device, dtype=torch.float32) + float(shift[0])) / H
    ww = (torch.arange(W, device=device, dtype=torch.float32) + float(shift[1])) / W
    out = torch.zeros((H, W, D), device=device, dtype=torch.float32)
    for j in range(params["a"].shape[0]):
        a, u, v, phi = (_t(params[k][j], device) for k in ("a", "u", "v", "phi"))
        arg = TWO_PI * (hh[:, None, None] * u + ww[None, :, None] * v) + phi
        out += a * torch.cos(arg)
    return out


def smooth_field_1d(N, D, seed, ncos=16, fmax=8.0, device="cpu") -> torch.Tensor:
    """[N,D] float32: per channel a sum of `ncos` random cosines along the sequence,
    frequencies U(0,fmax) cycles per sequence."""
    r = _rng(seed)
    a, u, phi = r.standard_normal((ncos, D)), r.uniform(0, fmax, (ncos, D)), r.uniform(0, TWO_PI, (ncos, D))
    nn = torch.arange(N, device=device, dtype=torch.float32) / N
    out = torch.zeros((N, D), device=device, dtype=torch.float32)
    for j in range(ncos):
        out += _t(a[j], device) * torch.cos(TWO_PI * nn[:, None] * _t(u[j], device) + _t(phi[j], device))
    return out


def _scale_outliers(x2d: torch.Tensor, frac: float, seed: int) -> torch.Tensor:
    """Multiply a seeded `frac` of the rows of x2d [T,D] by 10 (high-norm outlier tokens)."""
    T = x2d.shape[0]
    k = max(1, int(round(frac * T)))
    pos = _rng(seed + 77).choice(T, size=k, replace=False)
    x2d[torch.as_tensor(np.sort(pos), device=x2d.device)] *= 10.0
    return x2d


def _cast(x: torch.Tensor, dtype: str) -> torch.Tensor:
    return x.to(torch.bfloat16) if dtype == "bf16" else x.to(torch.float32)


def oim_input(config: int, device="cpu", batch=None, hw=None, dim=None) -> torch.Tensor:
    """Visual-encoder tokens [B,H,W,D] of one configuration (dtype as the configuration says).
    `batch`, `hw`, `dim` shrink the case for CPU-sized tests; the recipe stays the same."""
    c = CONFIGS[config]
    B = batch or c["B"]
    H, W = hw or (c["H"], c["W"])
    D = dim or c["D"]
    imgs = []
    if config == 3:
        frames = c["frames"]
        for b in range(B):
            video, t = divmod(b, frames)
            seed = 1000 * config + video
            r = _rng(seed)
            params = dict(a=r.standard_normal((8, D)), u=r.uniform(-2, 2, (8, D)),
                          v=r.uniform(-2, 2, (8, D)), phi=r.uniform(0, TWO_PI, (8, D)))
            drift = r.uniform(-0.5, 0.5, 2)
            x = smooth_field_2d(H, W, D, seed, device=device, shift=(t * drift[0], t * drift[1]), params=params)
            x += _noise((H, W, D), 0.05, 100000 * config + b, device)
            imgs.append(x)
    else:
        for b in range(B):
            seed = 1000 * config + b
            x = smooth_field_2d(H, W, D, seed, device=device)
            if config == 2:
                r = _rng(seed + 31)
                for _ in range(4):
                    sh = int(r.uniform(H / 8, H / 2)); sw = int(r.uniform(W / 8, W / 2))
                    h0 = int(r.integers(0, H - sh + 1)); w0 = int(r.integers(0, W - sw + 1))
                    x[h0:h0 + sh, w0:w0 + sw] += _t(2.0 * r.standard_normal(D), device)
            x += _noise((H, W, D), 0.1, seed, device)
            if config == 1:
                _scale_outliers(x.view(H * W, D), 0.02, seed)
            imgs.append(x)
    return _cast(torch.stack(imgs), c["dtype"])


def projection(D_in: int, D_out: int, seed: int, device="cpu") -> torch.Tensor:
    """Seeded N(0, 1/sqrt(D_in)) matrix standing in for the projector and the first LLM layers."""
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) + 0xBEEF)
    return torch.randn((D_in, D_out), generator=g, device=device, dtype=torch.float32) / math.sqrt(D_in)


def spu_input_from_tokens(config: int, merged: torch.Tensor, dim_out=None) -> torch.Tensor:
    """LLM-side hidden states for configurations 0-3: the merged visual tokens [B,T,D] times the
    seeded projection; configuration 3 concatenates the frames of each video in time order."""
    c = CONFIGS[config]
    D_out = dim_out or c["D_llm"]
    P = projection(merged.shape[-1], D_out, 1000 * config + 7, merged.device)
    y = merged.to(torch.float32) @ P
    if config == 3:
        frames = c["frames"]
        if y.shape[0] % frames == 0:
            y = y.reshape(y.shape[0] // frames, frames * y.shape[1], D_out)
    return _cast(y, c["dtype"])


def spu_stress_input(device="cpu", batch=None, n_tokens=None, dim=None) -> torch.Tensor:
    """Configuration 4's SPU input [B,N,D] bf16: smooth 1D field + N(0,0.2) noise + 1% outlier tokens."""
    c = CONFIGS[4]
    B, N, D = batch or c["spu_B"], n_tokens or c["spu_N"], dim or c["D_llm"]
    seqs = []
    for b in range(B):
        seed = 4000 + 100 + b
        x = smooth_field_1d(N, D, seed, device=device)
        x += _noise((N, D), 0.2, seed, device)
        _scale_outliers(x, 0.01, seed)
        seqs.append(x.to(torch.bfloat16))
    return torch.stack(seqs)


def keep_count(ratio: float, N: int) -> int:
    return int(math.floor(ratio * N + 0.5))
