"""Seeded synthetic inputs shaped like Stable Diffusion v1.4 UNet layer tensors.

This module only draws random tensors. It holds none of the quantization
method's arithmetic, so the CPU oracle tests and the CUDA path can both take
their inputs from it and still share no code of the method itself.

Recipe (all draws from numpy's PCG64 `default_rng((seed, tensor_id))`):

* activations  X[t, c] = z[t, c] * cs[c] * ts[t mod P],  z ~ N(0, 1), stored fp16.
  `cs[c]` is 30 for a seeded choice of outlier channels and 1 elsewhere;
  `ts[p]` is 20 for a seeded choice of outlier pixel (token) positions and 1
  elsewhere.  The outlier positions depend on `seed` only, so a calibration
  draw (another `tensor_id`) has its outliers in the same places, which is the
  behaviour the paper reports (Sec. 3.2: outliers sit on a few fixed channels
  or pixels and stay there when prompts and seeds change).
* weights ~ N(0, 0.02^2), bias ~ N(0, 0.01^2), stored fp16.
* cross-attention: Q ~ N(0,1); context ~ N(0,1) [B, 77, 768] projected with
  W ~ N(0, 0.02^2) to K and V; the <start> key gets a logit bias of about +6
  through the last feature (Q[..., d-1] = 1, K[b, 0, h, d-1] = 6 sqrt(d),
  K[b, j>=1, h, d-1] = 0) so column 0 of the softmax dominates as in Fig. 5(a).
"""
from __future__ import annotations

import math

import numpy as np

CH_OUTLIER_GAIN = 30.0
TOK_OUTLIER_GAIN = 20.0


def _rng(seed: int, tensor_id: int) -> np.random.Generator:
    return np.random.default_rng((int(seed), int(tensor_id)))


def outlier_channels(seed: int, C: int, n: int | None = None) -> np.ndarray:
    """Sorted indices of the outlier channels (1% of C, rounded up, unless n is given)."""
    if n is None:
        n = int(math.ceil(0.01 * C))
    perm = _rng(seed, 900_001).permutation(C)
    return np.sort(perm[:n])


def outlier_tokens(seed: int, P: int, n: int | None = None) -> np.ndarray:
    """Sorted indices of the outlier pixel positions (0.5% of P, at least one)."""
    if n is None:
        n = max(1, int(round(0.005 * P)))
    perm = _rng(seed, 900_002).permutation(P)
    return np.sort(perm[:n])


def activations(seed: int, tensor_id: int, n_samples: int, P: int, C: int,
                n_out_ch: int | None = None, n_out_tok: int | None = None,
                token_outliers: bool = True) -> np.ndarray:
    """fp16 activation matrix [n_samples * P, C] with channel and pixel outliers."""
    z = _rng(seed, tensor_id).standard_normal((n_samples * P, C), dtype=np.float32)
    cs = np.ones(C, dtype=np.float32)
    cs[outlier_channels(seed, C, n_out_ch)] = CH_OUTLIER_GAIN
    z *= cs[None, :]
    if token_outliers:
        ts = np.ones(P, dtype=np.float32)
        ts[outlier_tokens(seed, P, n_out_tok)] = TOK_OUTLIER_GAIN
        z *= np.tile(ts, n_samples)[:, None]
    return z.astype(np.float16)


def weights(seed: int, tensor_id: int, N: int, K: int, std: float = 0.02) -> np.ndarray:
    """fp16 weight matrix [N, K] ~ N(0, std^2)."""
    w = _rng(seed, tensor_id).standard_normal((N, K), dtype=np.float32) * np.float32(std)
    return w.astype(np.float16)


def bias(seed: int, tensor_id: int, N: int, std: float = 0.01) -> np.ndarray:
    b = _rng(seed, tensor_id).standard_normal(N, dtype=np.float32) * np.float32(std)
    return b.astype(np.float16)


def conv_weights(seed: int, tensor_id: int, N: int, C: int, std: float = 0.02) -> np.ndarray:
    """fp16 3x3 filter bank [N, 3, 3, C] (out channel, ky, kx, in channel)."""
    w = _rng(seed, tensor_id).standard_normal((N, 3, 3, C), dtype=np.float32) * np.float32(std)
    return w.astype(np.float16)


def attention_inputs(seed: int, B: int, H: int, nq: int, nk: int, d: int,
                     ctx_dim: int = 768, start_bias: float = 6.0):
    """fp16 Q [B, nq, H, d] and K, V [B, nk, H, d] for cross-attention."""
    rq = _rng(seed, 910_001)
    Q = rq.standard_normal((B, nq, H * d), dtype=np.float32)
    ctx = _rng(seed, 910_002).standard_normal((B, nk, ctx_dim)).astype(np.float64)
    Wk = _rng(seed, 910_003).standard_normal((H * d, ctx_dim)) * 0.02
    Wv = _rng(seed, 910_004).standard_normal((H * d, ctx_dim)) * 0.02
    K = ctx @ Wk.T
    V = ctx @ Wv.T
    Q = Q.reshape(B, nq, H, d)
    K = K.reshape(B, nk, H, d)
    V = V.reshape(B, nk, H, d)
    Q[..., d - 1] = 1.0
    K[:, 0, :, d - 1] = start_bias * math.sqrt(d)
    K[:, 1:, :, d - 1] = 0.0
    return Q.astype(np.float16), K.astype(np.float16), V.astype(np.float16)
