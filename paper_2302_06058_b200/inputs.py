"""Seeded synthetic inputs for the Bi-Mask layer step.

This module only draws numbers: it holds none of the method's arithmetic, so both the
CUDA path's tests/benchmark and the CPU oracle's tests may use it.

The shapes stand in for the models the paper trains (ResNet-50 3x3 convolutions as
im2col matrices, DeiT-small block linears) plus a large MLP pair as a roofline stress
case.  Weights are i.i.d. normal with the usual initialisation scale, activations and
output gradients are N(0, 1) rounded to bfloat16.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch


@dataclass(frozen=True)
class Layer:
    I: int      # output rows of W
    J: int      # input dim of W
    T: int      # tokens (rows of X and dY)


@dataclass(frozen=True)
class Config:
    name: str
    layers: tuple
    N: int
    M: int
    P: int              # number of candidate permutations (the paper's K)
    init: str           # "kaiming" or "trunc"


_RESNET = (Layer(64, 576, 32 * 56 * 56), Layer(128, 1152, 32 * 28 * 28),
           Layer(256, 2304, 32 * 14 * 14), Layer(512, 4608, 32 * 7 * 7))
_DEIT = (Layer(1152, 384, 64 * 197), Layer(384, 384, 64 * 197),
         Layer(1536, 384, 64 * 197), Layer(384, 1536, 64 * 197))

CONFIGS = {
    1: Config("single-256", (Layer(256, 256, 128),), 2, 4, 8, "kaiming"),
    2: Config("resnet50-2:4", _RESNET, 2, 4, 32, "kaiming"),
    3: Config("deit-small-2:4", _DEIT, 2, 4, 32, "trunc"),
    4: Config("resnet50-1:4", _RESNET, 1, 4, 64, "kaiming"),
    5: Config("mlp-16k-2:4", (Layer(16384, 4096, 8192), Layer(4096, 16384, 8192)), 2, 4, 128, "kaiming"),
}


def perm_seed(cfg: int) -> int:
    return 42 + cfg


def _gen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return g


def make_weight(I: int, J: int, seed: int, init: str = "kaiming") -> np.ndarray:
    """fp32 I x J weight.  kaiming: N(0, 2/J).  trunc: N(0, 0.02^2) truncated at +-2."""
    if init == "kaiming":
        W = torch.randn(I, J, generator=_gen(seed), dtype=torch.float32) * float(np.sqrt(2.0 / J))
    elif init == "trunc":
        W = torch.empty(I, J, dtype=torch.float32)
        torch.nn.init.trunc_normal_(W, mean=0.0, std=0.02, a=-2.0, b=2.0, generator=_gen(seed))
    else:
        raise ValueError(init)
    return W.numpy()


def make_activation(T: int, C: int, seed: int) -> np.ndarray:
    """N(0,1) rounded to bfloat16; returned as uint16 bit patterns, T x C."""
    x = torch.randn(T, C, generator=_gen(seed), dtype=torch.float32).to(torch.bfloat16)
    return x.view(torch.int16).numpy().view(np.uint16)


def make_layer(cfg: int, layer: int, T: int | None = None):
    """(W fp32 I x J, X bf16-bits T x J, dY bf16-bits T x I) for layer `layer` of config `cfg`.

    Seeds: 1000*cfg + 10*layer + r with r = 0 (W), 1 (X), 2 (dY).  T may be overridden to
    take a token slice of the same stream shape (used for bounded CPU timing)."""
    c = CONFIGS[cfg]
    L = c.layers[layer]
    T = L.T if T is None else T
    base = 1000 * cfg + 10 * layer
    W = make_weight(L.I, L.J, base + 0, c.init)
    X = make_activation(T, L.J, base + 1)
    dY = make_activation(T, L.I, base + 2)
    return W, X, dY


def planted_transposable(I: int, J: int, N: int, M: int, seed: int):
    """Weights whose forward N:M mask is also N:M along every aligned column block, with
    the rows then scrambled by a random permutation Q.

    Construction: tile an M x M circulant pattern (row r keeps columns r, r+1, .., r+N-1
    mod M), give kept positions magnitudes in [1, 2) and the others magnitudes in
    (0, 0.5), random signs.  Returns (W_scrambled, Q_inverse) where row k of
    W_scrambled[Q_inverse] is row k of the unscrambled matrix."""
    rng = np.random.default_rng(seed)
    r = np.arange(I)[:, None] % M
    c = np.arange(J)[None, :] % M
    kept = ((c - r) % M) < N
    mag = np.where(kept, 1.0 + rng.random((I, J)), 0.5 * rng.random((I, J)) + 1e-3)
    W = (mag * rng.choice([-1.0, 1.0], size=(I, J))).astype(np.float32)
    Q = rng.permutation(I)
    Ws = np.empty_like(W)
    Ws[Q, :] = W            # unscrambled row k lands at row Q[k]  => Ws[Q] == W
    return Ws, Q.astype(np.int32)
