"""Seeded synthetic inputs for the DiRotQ linear layer.

This module only *makes inputs*: activations with planted outlier channels and a
shared low-rank component, a calibration batch, the per-layer rotation built from
it, and random weights.  It holds none of the layer's arithmetic (no quantizer,
no fold, no GEMM); both the CPU oracle and the CUDA library are handed the very
same arrays produced here.

What stands in for what: the paper calibrates on activations of pretrained
PixArt-Sigma / FLUX.1-dev (Sec. 5.1, App. B), which are not available offline.
The generator reproduces their *shape*: a few channels with very large gain
(Fig. 1 reports max/median of 83x) on top of a low-rank shared component.

Rotation recipe (Sec. 4.2, App. B): second moment of the calibration batch,
eigenvectors sorted by decreasing eigenvalue, the first ``r`` kept as ``U_h``,
the rest multiplied by a data-independent random orthogonal ``R``;
``Q = [U_h, U_l R]``.
"""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

__all__ = [
    "LayerSpec", "PIXART", "FLUX", "bf16_bits", "bf16_bits_to_f32", "make_tokens",
    "make_rotation", "make_weights", "make_layer_inputs",
]


@dataclasses.dataclass(frozen=True)
class ActivationModel:
    """Structure of the synthetic activations of one model family."""
    name: str
    n_outliers: int   # number of planted outlier channels
    gain: float       # their gain over the ordinary channels
    rho: int          # rank of the shared component


PIXART = ActivationModel("pixart", 8, 50.0, 16)
FLUX = ActivationModel("flux", 16, 80.0, 32)


@dataclasses.dataclass(frozen=True)
class LayerSpec:
    K: int
    N: int
    r: int = 32
    G: int = 64
    model: ActivationModel = PIXART
    seed: int = 0
    calib_tokens: int = 2048

    @property
    def K_l(self) -> int:
        return self.K - self.r

    @property
    def n_g(self) -> int:
        return -(-self.K_l // self.G)


def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=np.random.SeedSequence(list(key)).generate_state(2, dtype=np.uint64)))


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float64/float32 values to bfloat16 (nearest, ties to even); returns uint16 bit patterns.

    Input preparation only (the library's inputs *are* bf16 tensors)."""
    a64 = np.asarray(a, dtype=np.float64)
    f = a64.astype(np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    down = (bits & 0xFFFF0000).astype(np.uint32)
    # neighbour one bf16 step away from zero in magnitude
    up = (down.astype(np.uint64) + 0x10000).astype(np.uint32)
    d_lo = np.abs(a64 - down.view(np.float32).astype(np.float64))
    with np.errstate(over="ignore", invalid="ignore"):
        d_hi = np.abs(a64 - up.view(np.float32).astype(np.float64))
    take_up = (d_hi < d_lo) | ((d_hi == d_lo) & (((down >> 16) & 1) == 1))
    out = np.where(take_up, up, down)
    return (out >> 16).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def _layer_stats(spec: LayerSpec):
    g = _rng(spec.seed, spec.K, 11)
    m = spec.model
    outliers = g.choice(spec.K, size=m.n_outliers, replace=False)
    gain = np.ones(spec.K)
    gain[outliers] = m.gain
    basis = g.standard_normal((m.rho, spec.K))
    return outliers, gain, basis


def make_tokens(spec: LayerSpec, T: int, batch_seed: int) -> np.ndarray:
    """``T`` tokens ``x = z*gain + (3/sqrt(rho)) A B`` rounded to bf16; returns uint16 bits [T, K]."""
    _, gain, basis = _layer_stats(spec)
    g = _rng(spec.seed, spec.K, 23, batch_seed)
    out = np.empty((T, spec.K), dtype=np.uint16)
    step = max(1, (1 << 24) // spec.K)
    for t0 in range(0, T, step):
        t1 = min(T, t0 + step)
        z = g.standard_normal((t1 - t0, spec.K))
        a = g.standard_normal((t1 - t0, spec.model.rho))
        out[t0:t1] = bf16_bits(z * gain + (3.0 / np.sqrt(spec.model.rho)) * (a @ basis))
    return out


def make_rotation(spec: LayerSpec, device: str = "cpu") -> np.ndarray:
    """Rotation ``Q = [U_h, U_l R]`` in float64, [K, K]; column j is basis vector j.

    ``device`` only selects where torch runs the eigendecomposition / QR / product
    (float64 either way)."""
    K, r = spec.K, spec.r
    xc = bf16_bits_to_f32(make_tokens(spec, spec.calib_tokens, batch_seed=1_000_003)).astype(np.float64)
    X = torch.from_numpy(xc).to(device)
    sigma = (X.T @ X) / float(spec.calib_tokens)
    # damping: a multiple of the identity, leaves the eigenvectors unchanged
    sigma += 0.01 * torch.mean(torch.diagonal(sigma)) * torch.eye(K, dtype=torch.float64, device=device)
    evals, evecs = torch.linalg.eigh(sigma)
    order = torch.argsort(evals, descending=True, stable=True)
    U = evecs[:, order]
    # sign convention: largest-magnitude entry of every eigenvector is positive
    idx = torch.argmax(U.abs(), dim=0)
    sgn = torch.sign(U[idx, torch.arange(K, device=device)])
    sgn[sgn == 0] = 1.0
    U = U * sgn
    K_l = K - r
    gr = _rng(K_l, 37)  # one R per residual dimension, data independent (Sec. 4.2)
    Gm = torch.from_numpy(gr.standard_normal((K_l, K_l))).to(device)
    Qr, Rr = torch.linalg.qr(Gm)
    d = torch.sign(torch.diagonal(Rr))
    d[d == 0] = 1.0
    R = Qr * d
    Q = torch.cat([U[:, :r], U[:, r:] @ R], dim=1)
    return Q.cpu().numpy()


def make_weights(spec: LayerSpec, with_bias: bool = True):
    """``W ~ N(0, 0.02^2)`` float32 [K, N]; bias bf16 bits [N] (or None)."""
    g = _rng(spec.seed, spec.K, spec.N, 41)
    W = (0.02 * g.standard_normal((spec.K, spec.N))).astype(np.float32)
    bias = bf16_bits(0.02 * g.standard_normal(spec.N)) if with_bias else None
    return W, bias


def make_layer_inputs(spec: LayerSpec, M: int, batch_seed: int = 7, device: str = "cpu", with_bias: bool = True):
    """All inputs of one layer call: dict with x (bf16 bits), Q (f64), W (f32), bias (bf16 bits)."""
    W, bias = make_weights(spec, with_bias)
    return {
        "x": make_tokens(spec, M, batch_seed),
        "Q": make_rotation(spec, device=device),
        "W": W,
        "bias": bias,
    }
