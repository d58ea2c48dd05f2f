"""Seeded synthetic inputs for the mixed-precision linear layer.

This module only draws random numbers and names layer shapes.  It holds none of
the method's arithmetic (no salience, no quantizer, no packing): the CUDA path
and the CPU checker both start from the arrays produced here.

The arrays stand in for the LLaMA checkpoints the paper deploys (Sec. 4.3 and
the deployment tables): only the layer shapes and the qualitative structure the
paper describes are kept -- near-Gaussian weights whose salience is driven by a
few outlier input channels (Theorem 1, Sec. 3.2.1).

Recipe (per layer, all draws from numpy PCG64 streams derived from a seed tuple):
  W   fp16 [N][K]  N(0, 0.02^2) drawn in fp32; round(0.01*K) distinct columns,
                   chosen uniformly, are multiplied by 10 before rounding to fp16
  a   fp32 [K]     exp(N(0,1)): per-input-channel activation norms (lognormal)
  x   fp16 [M][K]  N(0,1)
"""
from __future__ import annotations

import numpy as np

GROUP = 128

# (name, N = out_features, K = in_features) for one transformer block
LAYER_SETS = {
    "llama-7b": [("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
                 ("gate", 11008, 4096), ("up", 11008, 4096), ("down", 4096, 11008)],
    "llama-13b": [("q", 5120, 5120), ("k", 5120, 5120), ("v", 5120, 5120), ("o", 5120, 5120),
                  ("gate", 13824, 5120), ("up", 13824, 5120), ("down", 5120, 13824)],
    "llama-2-70b": [("q", 8192, 8192), ("k", 1024, 8192), ("v", 1024, 8192), ("o", 8192, 8192),
                    ("gate", 28672, 8192), ("up", 28672, 8192), ("down", 8192, 28672)],
}
N_BLOCKS = {"llama-7b": 32, "llama-13b": 40, "llama-2-70b": 80}

_STREAM_W, _STREAM_COLS, _STREAM_A, _STREAM_X = 0, 1, 2, 3


def _name_key(name: str) -> int:
    key = 0
    for ch in name.encode():
        key = (key * 131 + ch) % (2**31 - 1)
    return key


def layer_seed(model: str, layer: str, block: int, base_seed: int = 2405_14917) -> tuple:
    """Seed tuple of one layer: (base, model key, layer key, block index)."""
    return (int(base_seed), _name_key(model), _name_key(layer), int(block))


def _rng(seed: tuple, stream: int, extra: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence(list(seed) + [stream, extra])))


def make_weight(seed: tuple, N: int, K: int, outlier_frac: float = 0.01, outlier_gain: float = 10.0,
                sigma: float = 0.02) -> np.ndarray:
    """fp16 weight matrix [N][K] with a few amplified input columns."""
    w = _rng(seed, _STREAM_W).standard_normal((N, K), dtype=np.float32)
    w *= np.float32(sigma)
    n_out = int(round(outlier_frac * K))
    if n_out > 0:
        cols = _rng(seed, _STREAM_COLS).choice(K, size=n_out, replace=False)
        w[:, cols] *= np.float32(outlier_gain)
    return w.astype(np.float16)


def make_act_norms(seed: tuple, K: int) -> np.ndarray:
    """fp32 [K] lognormal(0, 1) per-channel activation norms."""
    return np.exp(_rng(seed, _STREAM_A).standard_normal(K)).astype(np.float32)


def make_x(seed: tuple, M: int, K: int) -> np.ndarray:
    """fp16 activations [M][K] ~ N(0, 1)."""
    return _rng(seed, _STREAM_X, M).standard_normal((M, K), dtype=np.float32).astype(np.float16)


def make_calibration_x(seed: tuple, T: int, K: int, rank: int = 16, mix: float = 0.7) -> np.ndarray:
    """fp16 calibration activations [T][K] with correlated channels: every token is a mixture of
    `rank` shared directions plus independent noise, scaled per channel by the lognormal activation
    norms (so a few channels dominate, as in the outlier channels of LLM activations)."""
    r = _rng(seed, _STREAM_X, 7000 + T)
    basis = r.standard_normal((rank, K))
    coeff = r.standard_normal((T, rank))
    noise = r.standard_normal((T, K))
    x = mix * (coeff @ basis) / np.sqrt(rank) + (1.0 - mix) * noise
    x *= make_act_norms(seed, K).astype(np.float64)
    return x.astype(np.float16)


def model_layers(model: str, n_blocks: int | None = None):
    """Yield (layer name, block, N, K, seed) over n_blocks blocks of a model."""
    nb = N_BLOCKS[model] if n_blocks is None else n_blocks
    for blk in range(nb):
        for (name, N, K) in LAYER_SETS[model]:
            yield name, blk, N, K, layer_seed(model, name, blk)


def algorithmic_bytes(M: int, N: int, K: int, bits) -> int:
    """Bytes one call must move: packed codes + fp16 scales and zeros + bit map + x + y."""
    bits = np.asarray(bits, dtype=np.int64)
    G = K // GROUP
    assert bits.shape == (G,)
    return int(N * GROUP * int(bits.sum()) // 8 + 2 * 2 * G * N + G + 2 * M * K + 2 * M * N)


def make_weight_and_norms_device(seed: tuple, N: int, K: int, device, outlier_frac: float = 0.01,
                                 outlier_gain: float = 10.0, sigma: float = 0.02):
    """Same recipe as make_weight / make_act_norms, drawn on the device with torch's seeded generator.

    Used where hundreds of full-size layers are needed (billions of draws); the values differ
    from the NumPy streams but follow the same distributions.  Returns (W fp16 [N][K], a fp32 [K]).
    """
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(int(np.random.SeedSequence(list(seed)).generate_state(1, dtype=np.uint64)[0] >> 1))
    w = torch.randn((N, K), generator=gen, device=device, dtype=torch.float32) * sigma
    n_out = int(round(outlier_frac * K))
    if n_out > 0:
        cols = torch.randperm(K, generator=gen, device=device)[:n_out]
        w[:, cols] *= outlier_gain
    a = torch.exp(torch.randn(K, generator=gen, device=device, dtype=torch.float32))
    return w.to(torch.float16), a
