"""Cross-attention with log2-quantized softmax scores, Sec. 3.3 (Eq. 3, Eq. 8, Eq. 9).

Test infrastructure only; see the package docstring.
"""
from __future__ import annotations

import numpy as np

from .quantizers import log_quantize, log_dequantize, group_params_array, quantize_canonical_f32

PER_PROMPT, PER_PROMPT_HEAD, PER_CALL = 0, 1, 2
FLT_MIN = float(np.finfo(np.float32).tiny)


def softmax_scores(Q, K):
    """Eq. 3: A = softmax_j(Q_i . K_j / sqrt(d)), fp64.  Q [B, nq, H, d], K [B, nk, H, d] -> A [B, H, nq, nk]."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    d = Q.shape[-1]
    logits = np.einsum("bqhd,bkhd->bhqk", Q, K) / np.sqrt(np.float64(d))
    logits -= logits.max(axis=-1, keepdims=True)
    e = np.exp(logits)
    return e / e.sum(axis=-1, keepdims=True)


def prompt_scale(A, gran=PER_PROMPT):
    """The dynamic scale of Eq. 8: s = max(A[:, 1:]), the largest score off the <start> column.

    Eq. 8 writes A as one n_q x n_k map while the text ties the scale to the
    input prompt; reading (parity unpinned): PER_PROMPT takes the maximum over
    all heads, queries and keys j >= 1 of one prompt.  PER_PROMPT_HEAD and
    PER_CALL are the narrower and wider scopes.  Returns s broadcastable to A
    [B, H, nq, nk]; a zero maximum is raised to the smallest normal fp32.
    """
    rest = A[..., 1:]
    if gran == PER_PROMPT:
        s = rest.max(axis=(1, 2, 3), keepdims=True)
    elif gran == PER_PROMPT_HEAD:
        s = rest.max(axis=(2, 3), keepdims=True)
    else:
        s = rest.max(keepdims=True)
    return np.maximum(s, FLT_MIN)


def quantize_values(V, v_bits):
    """V_hat of Eq. 9 when the value operand is quantized too.

    The paper names V_hat "quantized value" without giving its quantizer; reading (parity unpinned): the
    linear quantizer of Eq. 1 with the range of Eq. 6 taken over one head's [n_k, d] slab of one prompt,
    code decided in fp32 (`quantize_canonical_f32`), de-quantized as s (q - Z) in fp32.  Rows j >= 1 are
    the fp16 operand of the product and are rounded to fp16; row 0 (the <start> value, which meets a
    full-precision score) stays fp32.  V [B, nk, H, d] -> (V_hat fp64 [B, nk, H, d], codes, s [B, H], Z [B, H]).
    """
    V32 = np.asarray(V, dtype=np.float32)
    lo = V32.min(axis=(1, 3))
    hi = V32.max(axis=(1, 3))
    s, inv_s, Z = group_params_array(lo, hi, v_bits)                          # [B, H]
    codes = quantize_canonical_f32(V32, inv_s[:, None, :, None], Z[:, None, :, None], v_bits)
    deq = (s[:, None, :, None] * (codes - Z[:, None, :, None]).astype(np.float32)).astype(np.float32)
    V_hat = deq.astype(np.float64)
    V_hat[:, 1:] = deq[:, 1:].astype(np.float16).astype(np.float64)
    return V_hat, codes, s, Z


def cross_attn_logq(Q, K, V, bits, gran=PER_PROMPT, fixed_scale=None, v_bits=None):
    """Attention-aware quantization (Eq. 8, Eq. 9), fp64 throughout.

    Steps in the paper's order: full-precision softmax (Eq. 3); scale s from the
    scores off the <start> column (or `fixed_scale`, the static variant of the
    ablation in Table 3(c)); log2 codes of columns j >= 1 (Eq. 8, which is Eq. 2
    with that s); A_hat = [A[:, 0], s 2^-codes] with column 0 untouched; the
    product A_hat V as the sum of the <start> term and the quantized rest
    (Eq. 9).  No re-normalisation of A_hat (none is described).  V stays as
    given (V_hat = V) unless `v_bits` is set, in which case V_hat =
    `quantize_values(V, v_bits)`.  Returns O [B, nq, H, d], codes
    [B, H, nq, nk-1], s (broadcast shape), A.
    """
    A = softmax_scores(Q, K)
    V = np.asarray(V, dtype=np.float64) if v_bits is None else quantize_values(V, v_bits)[0]
    if A.shape[-1] < 2:
        raise ValueError("n_k < 2: no score off the <start> column to scale by")
    if fixed_scale is None:
        s = prompt_scale(A, gran)
    else:
        s = np.maximum(np.asarray(fixed_scale, dtype=np.float64).reshape(-1, 1, 1, 1), FLT_MIN)
    s_full = np.broadcast_to(s, A.shape[:-1] + (1,))
    codes = log_quantize(A[..., 1:], s_full, bits)
    return split_product(A, codes, s, V), codes, s, A


def split_product(A, codes, s, V):
    """Eq. 9: A_hat V = A[:, 0] V[0] + (s 2^-codes) V[1:], fp64, for given codes [B, H, nq, nk-1]."""
    V = np.asarray(V, dtype=np.float64)
    s_full = np.broadcast_to(s, A.shape[:-1] + (1,))
    A_hat_rest = log_dequantize(codes, s_full)
    return (np.einsum("bhq,bhd->bqhd", A[..., 0], V[:, 0])
            + np.einsum("bhqk,bkhd->bqhd", A_hat_rest, V[:, 1:]))


def attention_reference(Q, K, V):
    """Plain softmax attention softmax(Q K^T / sqrt(d)) V in fp64 (no quantization)."""
    A = softmax_scores(Q, K)
    return np.einsum("bhqk,bkhd->bqhd", A, np.asarray(V, dtype=np.float64))


def self_attn_logq(Q, K, V, bits, fixed_scale=None):
    """Log2-quantized attention scores without a <start> column (self-attention, Sec. 3.3: the log
    quantizer of Eq. 2 is applied "to both self and cross-attentions"), fp64 throughout.

    A = softmax(Q K^T / sqrt(d)) (Eq. 3); codes = clamp(rint(-log2(A / s)), 0, 2^b - 1) over ALL keys
    (Eq. 2); A_hat = s 2^-codes; O = A_hat V.  The paper gives the dynamic scale only for
    cross-attention; reading (parity unpinned): s is the largest score of each query row unless
    `fixed_scale` ([B], one per prompt) is given.  No re-normalisation, V as given.
    Q [B, nq, H, d], K, V [B, nk, H, d] -> O [B, nq, H, d], codes [B, H, nq, nk], s (broadcast shape), A.
    """
    A = softmax_scores(Q, K)
    V = np.asarray(V, dtype=np.float64)
    if fixed_scale is None:
        s = np.maximum(A.max(axis=-1, keepdims=True), FLT_MIN)
    else:
        s = np.maximum(np.asarray(fixed_scale, dtype=np.float64).reshape(-1, 1, 1, 1), FLT_MIN)
    s_full = np.broadcast_to(s, A.shape[:-1] + (1,))
    codes = log_quantize(A, s_full, bits)
    return self_product(codes, s, V), codes, s, A


def self_product(codes, s, V):
    """O = (s 2^-codes) V for given codes [B, H, nq, nk], fp64."""
    V = np.asarray(V, dtype=np.float64)
    s_full = np.broadcast_to(s, codes.shape[:-1] + (1,))
    return np.einsum("bhqk,bkhd->bqhd", log_dequantize(codes, s_full), V)
