"""Group-quantized linear / 3x3 conv layer: Eq. 1 with Eq. 6 parameters, integer product, de-quantize.

Test infrastructure only; see the package docstring.

The paper states the quantizers (Eq. 1, Eq. 6) and counts the layer's cost as
integer multiply-accumulates (BOPs, Sec. 4.1) but never writes the integer
algebra out.  It follows from Eq. 1's right half x_dq = s (x_q - z) applied to
the activations of each group and w_dq = sw * wq for the weights:

    Y[t, o] = bias[o] + sw[o] * sum_g s[t, g] * ( acc_g[t, o] - Z[t, g] * wsum_g[o] )
    acc_g[t, o] = sum_{c in group g} x_q[t, c] * wq[o, c]        (int64)
    wsum_g[o]   = sum_{c in group g} wq[o, c]                    (int64)

with s, Z the parameters of the cell that row t and group g fall in.
"""
from __future__ import annotations

import numpy as np

from .quantizers import F32, group_params_array, quantize_canonical_f32


# --------------------------------------------------------------------------- weights
def weight_rtn(W, bits):
    """Per-out-channel symmetric round-to-nearest weight codes.

    Stands in for the paper's BRECQ / AdaRound weights (Sec. 4.1), which need a
    trained model.  fp32 sequence: sw = absmax / qmax, inv = 1 / sw,
    wq = clamp(rint(w * inv), -qmax, qmax), qmax = 2^(bits-1) - 1; an all-zero
    row gets sw = 1.  W is [N, ...]; the scale is per leading index.
    """
    W = np.asarray(W, dtype=F32)
    qmax = F32(2 ** (bits - 1) - 1)
    flat = W.reshape(W.shape[0], -1)
    absmax = np.max(np.abs(flat), axis=1).astype(F32)
    sw = np.where(absmax > 0, (absmax / qmax).astype(F32), F32(1.0)).astype(F32)
    inv = (F32(1.0) / sw).astype(F32)
    t = (flat * inv[:, None]).astype(F32)
    wq = np.clip(np.rint(t), -qmax, qmax).astype(np.int8)
    return wq.reshape(W.shape), sw


def pack_int4(wq):
    """Two's-complement 4-bit codes, two per byte along the last axis: low nibble = even index."""
    wq = np.asarray(wq, dtype=np.int8)
    assert wq.shape[-1] % 2 == 0
    u = wq.astype(np.uint8) & 0x0F
    return (u[..., 0::2] | (u[..., 1::2] << 4)).astype(np.uint8)


def unpack_int4(packed):
    """Inverse of `pack_int4`."""
    p = np.asarray(packed, dtype=np.uint8)
    lo = (p & 0x0F).astype(np.int16)
    hi = (p >> 4).astype(np.int16)
    lo = np.where(lo >= 8, lo - 16, lo)
    hi = np.where(hi >= 8, hi - 16, hi)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), dtype=np.int8)
    out[..., 0::2] = lo
    out[..., 1::2] = hi
    return out


# --------------------------------------------------------------------------- activations
def quantize_static(X, gr, timestep):
    """Eq. 1 with the calibrated cell parameters of `timestep` (Eq. 6, Eq. 7).

    Returns codes int32 [M, C] (original channel order) and the per-row
    parameter rows s [M, G], Z [M, G] that the de-quantizer needs.
    """
    X = np.asarray(X, dtype=F32)
    M = X.shape[0]
    r = np.asarray(gr.row_group)[np.arange(M) % gr.P]
    inv_rows = gr.inv_scale[timestep][r]          # [M, G]
    s_rows = gr.scale[timestep][r]
    z_rows = gr.zp[timestep][r]
    cg = np.asarray(gr.col_group)
    codes = quantize_canonical_f32(X, inv_rows[:, cg], z_rows[:, cg], gr.bits)
    return codes, s_rows, z_rows


def quantize_dynamic_token(X, col_group, G, bits):
    """Eq. 6 applied per token: the range of token t's members of channel group g.

    A per-token refinement of the paper's static tables (every token, and with it
    every outlier pixel, gets its own range per channel group).  Returns codes
    [M, C], s [M, G] float32, Z [M, G] int32.
    """
    X = np.asarray(X, dtype=F32)
    M = X.shape[0]
    cg = np.asarray(col_group)
    lo = np.zeros((M, G), dtype=F32)
    hi = np.zeros((M, G), dtype=F32)
    for g in range(G):
        cols = X[:, cg == g]
        if cols.shape[1]:
            lo[:, g], hi[:, g] = cols.min(axis=1), cols.max(axis=1)
    s, inv_s, Z = group_params_array(lo, hi, bits)
    codes = quantize_canonical_f32(X, inv_s[:, cg], Z[:, cg], bits)
    return codes, s, Z


# --------------------------------------------------------------------------- layer
def group_linear(codes, s_rows, z_rows, col_group, wq, sw, bias=None):
    """The layer formula of the module docstring for a linear layer; fp64 result [M, N]."""
    codes = np.asarray(codes, dtype=np.int64)
    wq64 = np.asarray(wq, dtype=np.int64)
    cg = np.asarray(col_group)
    G = s_rows.shape[1]
    Y = np.zeros((codes.shape[0], wq64.shape[0]), dtype=np.float64)
    for g in range(G):
        idx = np.flatnonzero(cg == g)
        if idx.size == 0:
            continue
        acc = codes[:, idx] @ wq64[:, idx].T                       # int64
        wsum = wq64[:, idx].sum(axis=1)                            # int64
        corr = acc - np.asarray(z_rows[:, g], dtype=np.int64)[:, None] * wsum[None, :]
        Y += np.asarray(s_rows[:, g], dtype=np.float64)[:, None] * corr.astype(np.float64)
    Y *= np.asarray(sw, dtype=np.float64)[None, :]
    if bias is not None:
        Y += np.asarray(bias, dtype=np.float64)[None, :]
    return Y


def group_conv3x3(codes, s_g, z_g, col_group, wq, sw, bias=None):
    """3x3, stride 1, zero-padding 1 convolution of the de-quantized activation.

    codes [n, H, W, C] (NHWC), one (s, Z) per channel group (static tables,
    channel dimension), wq [N, 3, 3, C].  A padded tap contributes exactly 0:
    the padding is a real zero of the de-quantized activation s (x_q - Z), so
    the integer sum runs over (x_q - Z) at in-image taps only.  Written as the
    sum over the nine taps of shifted products.  fp64 result [n, H, W, N].
    """
    codes = np.asarray(codes, dtype=np.int64)
    wq64 = np.asarray(wq, dtype=np.int64)
    n, H, W, C = codes.shape
    N = wq64.shape[0]
    cg = np.asarray(col_group)
    G = len(s_g)
    Y = np.zeros((n, H, W, N), dtype=np.float64)
    for g in range(G):
        idx = np.flatnonzero(cg == g)
        if idx.size == 0:
            continue
        centred = codes[..., idx] - int(z_g[g])                    # x_q - Z, int64
        acc = np.zeros((n, H, W, N), dtype=np.int64)
        for ky in range(3):
            for kx in range(3):
                dy, dx = ky - 1, kx - 1
                h0, h1 = max(0, -dy), min(H, H - dy)
                w0, w1 = max(0, -dx), min(W, W - dx)
                src = centred[:, h0 + dy:h1 + dy, w0 + dx:w1 + dx, :]
                acc[:, h0:h1, w0:w1, :] += src @ wq64[:, ky, kx, idx].T
        Y += np.float64(s_g[g]) * acc.astype(np.float64)
    Y *= np.asarray(sw, dtype=np.float64)
    if bias is not None:
        Y += np.asarray(bias, dtype=np.float64)
    return Y


def fake_quant_reference(codes, s_rows, z_rows, col_group, wq, sw, bias=None):
    """X_dq W_dq^T + bias from the de-quantized operands (Eq. 1 right half), fp64.

    An algebraically equal route to `group_linear` that never forms per-group
    integer sums; used to check the zero-point algebra.
    """
    cg = np.asarray(col_group)
    Xdq = np.asarray(s_rows, dtype=np.float64)[:, cg] * (
        np.asarray(codes, dtype=np.float64) - np.asarray(z_rows, dtype=np.float64)[:, cg])
    Wdq = np.asarray(sw, dtype=np.float64)[:, None] * np.asarray(wq, dtype=np.float64)
    Y = Xdq @ Wdq.T
    if bias is not None:
        Y += np.asarray(bias, dtype=np.float64)[None, :]
    return Y
