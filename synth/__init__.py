"""Seeded synthetic inputs for the LeanQuant per-linear-layer pass.

This module only draws random tensors.  It holds none of the method's
arithmetic (no Hessian, no grid, no quantisation) and is the one module that
both the float64 oracle's tests and the CUDA path's tests / benchmark import.

Every recipe is a stand-in for the paper's workloads (linear layers of
Llama-class models calibrated on 128 x 2048 tokens): the real weights and
calibration text are not available, so shapes, dtypes and value distributions
follow the benchmark configurations instead.

Notation follows Algorithm 1: ``W`` is r x c (r output rows, c input columns),
``X`` is c x n (feature-major, the n calibration tokens contiguous).

All draws come from a ``torch.Generator`` seeded per (seed, tensor name), so a
given (recipe, shape, seed, device type) always yields the same bits.  CPU and
CUDA generators are different streams: parity tests draw on the CPU and upload;
the benchmark draws on the device and downloads whatever sample the oracle needs.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, field

import torch

__all__ = ["Layer", "make_layer", "RECIPES", "CONFIGS", "config_layers"]


@dataclass
class Layer:
    """One synthetic linear layer: weights, calibration inputs and the settings
    the benchmark configuration attaches to it."""

    name: str
    W: torch.Tensor            # r x c
    X: torch.Tensor            # c x n, feature-major
    settings: dict = field(default_factory=dict)

    @property
    def r(self) -> int:
        return self.W.shape[0]

    @property
    def c(self) -> int:
        return self.W.shape[1]

    @property
    def n(self) -> int:
        return self.X.shape[1]


def _gen(seed: int, tag: str, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + zlib.crc32(tag.encode())) % (2**63 - 1))
    return g


def _randn(shape, g, device, dtype=torch.float32):
    return torch.randn(shape, generator=g, device=device, dtype=dtype)


# --------------------------------------------------------------------------- #
# weight recipes
# --------------------------------------------------------------------------- #
def weights_outlier_columns(r, c, seed, device, n_cols=4, factor=10.0, std=0.02):
    """N(0, std^2) weights with ``n_cols`` whole input columns scaled by ``factor``."""
    g = _gen(seed, "W", device)
    W = _randn((r, c), g, device) * std
    cols = torch.randperm(c, generator=_gen(seed, "Wcols", "cpu"))[:n_cols].to(device)
    W[:, cols] *= factor
    return W


def weights_outlier_entries(r, c, seed, device, frac=1e-3, factor=20.0, std=0.02):
    """N(0, std^2) weights with a fraction ``frac`` of single entries scaled by ``factor``."""
    g = _gen(seed, "W", device)
    W = _randn((r, c), g, device) * std
    mask = torch.rand((r, c), generator=_gen(seed, "Wmask", device), device=device) < frac
    W = torch.where(mask, W * factor, W)
    return W


# --------------------------------------------------------------------------- #
# calibration-input recipes (X is c x n); generated in column chunks so that the
# large configurations never hold more than one fp32 chunk besides the result
# --------------------------------------------------------------------------- #
def _channel_scales(c, seed, device, sigma=1.0, n_boost=0, boost=1.0):
    s = torch.exp(sigma * _randn((c,), _gen(seed, "Xscale", "cpu"), "cpu"))
    if n_boost:
        idx = torch.randperm(c, generator=_gen(seed, "Xboost", "cpu"))[:n_boost]
        s[idx] *= boost
    return s.to(device)


def inputs_scaled_gaussian(c, n, seed, device, dtype, n_boost=8, boost=50.0, chunk=16384):
    """Channel i ~ N(0, s_i^2), ln s ~ N(0,1), ``n_boost`` channels scaled by ``boost``."""
    s = _channel_scales(c, seed, device, 1.0, n_boost, boost)
    g = _gen(seed, "X", device)
    X = torch.empty((c, n), device=device, dtype=dtype)
    for j in range(0, n, chunk):
        m = min(chunk, n - j)
        X[:, j:j + m] = (_randn((c, m), g, device) * s[:, None]).to(dtype)
    return X


def inputs_low_rank(c, n, seed, device, dtype, rank=256, noise=0.05, chunk=16384):
    """(rank-``rank`` factor x coefficients + noise) x log-normal channel scales.

    The shared low-rank part makes channels strongly correlated, so H = 2XX^T is
    ill-conditioned and diag(H^-1) is heavy-tailed."""
    rank = min(rank, max(1, c // 4))
    s = _channel_scales(c, seed, device, 1.0)
    F = _randn((c, rank), _gen(seed, "XF", device), device) / rank ** 0.5
    g = _gen(seed, "X", device)
    X = torch.empty((c, n), device=device, dtype=dtype)
    for j in range(0, n, chunk):
        m = min(chunk, n - j)
        coef = _randn((rank, m), g, device)
        eps = _randn((c, m), g, device)
        X[:, j:j + m] = ((F @ coef + noise * eps) * s[:, None]).to(dtype)
    return X


def inputs_gated(c, n, seed, device, dtype, rank=64, chunk=16384):
    """SwiGLU-like activations: the product of two Gaussians (heavy-tailed), one of
    them carrying a low-rank shared component, times mild channel scales."""
    rank = min(rank, max(1, c // 4))
    s = _channel_scales(c, seed, device, 0.5)
    F = _randn((c, rank), _gen(seed, "XF", device), device) / rank ** 0.5
    g = _gen(seed, "X", device)
    X = torch.empty((c, n), device=device, dtype=dtype)
    for j in range(0, n, chunk):
        m = min(chunk, n - j)
        a = F @ _randn((rank, m), g, device) + 0.5 * _randn((c, m), g, device)
        b = _randn((c, m), g, device)
        X[:, j:j + m] = (a * b * s[:, None]).to(dtype)
    return X


RECIPES = {
    # name: (weight recipe, input recipe, dtype)
    "c1": (weights_outlier_columns, inputs_scaled_gaussian, torch.float32),
    "c2": (weights_outlier_entries, inputs_low_rank, torch.bfloat16),
    "c3": (weights_outlier_entries, inputs_gated, torch.bfloat16),
}


def make_layer(recipe: str, r: int, c: int, n: int, seed: int = 0, device="cpu",
               name: str | None = None, settings: dict | None = None,
               X: torch.Tensor | None = None) -> Layer:
    """Draw one layer.  ``X`` may be passed in for layers that share a Hessian."""
    wfn, xfn, dtype = RECIPES[recipe]
    W = wfn(r, c, seed, device).to(dtype)
    if X is None:
        X = xfn(c, n, seed, device, dtype)
    return Layer(name or recipe, W, X, dict(settings or {}))


# --------------------------------------------------------------------------- #
# the benchmark configurations (full sizes); ``scale`` shrinks every dimension
# for parity tests while keeping recipe and settings
# --------------------------------------------------------------------------- #
CONFIGS = {
    "c1": dict(recipe="c1", r=512, c=512, n=8192,
               settings=dict(grid="nonuniform", bits=4, p=4.0, block=128, n_iter=20, damp=0.01)),
    "c2": dict(recipe="c2", r=4096, c=4096, n=262144,
               settings=dict(grid="nonuniform", bits=4, p=4.0, block=128, n_iter=20, damp=0.01)),
    "c3": dict(recipe="c3", r=4096, c=14336, n=131072,
               settings=dict(grid="affine", bits=4, p=4.0, block=128, group=128, T=45, t=9, damp=0.01)),
}


def config_layers(name: str, seed: int = 0, device="cpu", scale: int = 1, n: int | None = None):
    """Layers of one benchmark configuration, dimensions divided by ``scale``."""
    cfg = CONFIGS[name]
    r, c = cfg["r"] // scale, cfg["c"] // scale
    n = n if n is not None else max(cfg["n"] // scale, 2 * c)
    return [make_layer(cfg["recipe"], r, c, n, seed, device, name=name, settings=cfg["settings"])]
