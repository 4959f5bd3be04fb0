"""Pins for the oracle's log-quantized cross-attention (Eq. 3, Eq. 8, Eq. 9)."""
import math

import numpy as np
import pytest

from oracle import attention as oa
from paper_2501_04304_b200 import synth


def _inputs(seed=0, B=2, H=2, nq=24, nk=9, d=8):
    return synth.attention_inputs(seed, B, H, nq, nk, d, ctx_dim=32)


def test_softmax_matches_library_sdpa():
    torch = pytest.importorskip("torch")
    Q, K, V = _inputs()
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q.astype(np.float64)).permute(0, 2, 1, 3),
        torch.from_numpy(K.astype(np.float64)).permute(0, 2, 1, 3),
        torch.from_numpy(V.astype(np.float64)).permute(0, 2, 1, 3)).permute(0, 2, 1, 3).numpy()
    got = oa.attention_reference(Q, K, V)
    assert np.max(np.abs(got - ref)) < 1e-12
    A = oa.softmax_scores(Q, K)
    assert np.allclose(A.sum(-1), 1.0, atol=1e-14)


def test_brute_force_tiny():
    Q, K, V = _inputs(seed=1, B=1, H=1, nq=16, nk=3, d=8)
    O, codes, s, A = oa.cross_attn_logq(Q, K, V, 8)
    Qf, Kf, Vf = Q.astype(float), K.astype(float), V.astype(float)
    P = [[0.0] * 3 for _ in range(16)]
    for i in range(16):
        l = [sum(Qf[0, i, 0, c] * Kf[0, j, 0, c] for c in range(8)) / math.sqrt(8) for j in range(3)]
        m = max(l)
        e = [math.exp(v - m) for v in l]
        P[i] = [v / sum(e) for v in e]
    smax = max(P[i][j] for i in range(16) for j in (1, 2))
    assert abs(float(s.ravel()[0]) - smax) < 1e-15
    for i in range(16):
        out = [P[i][0] * Vf[0, 0, 0, c] for c in range(8)]
        for j in (1, 2):
            q = min(max(round(-math.log2(P[i][j] / smax)), 0), 255)
            assert q == codes[0, 0, i, j - 1]
            for c in range(8):
                out[c] += smax * 2.0 ** -q * Vf[0, j, 0, c]
        assert np.allclose(O[0, i, 0], out, rtol=1e-12, atol=1e-15)


@pytest.mark.parametrize("bits", [4, 6, 8])
def test_structure_of_quantized_scores(bits):
    Q, K, V = _inputs(seed=2)
    B, nq, H, d = Q.shape
    nk = K.shape[1]
    O, codes, s, A = oa.cross_attn_logq(Q, K, V, bits)
    assert codes.min() >= 0 and codes.max() <= 2 ** bits - 1
    # the <start> column passes through unchanged: V = indicator of key 0 gives back A[:, 0] bit for bit
    V0 = np.zeros_like(V, dtype=np.float64); V0[:, 0] = 1.0
    O0, *_ = oa.cross_attn_logq(Q, K, V0, bits)
    assert np.array_equal(O0[..., 0], A[..., 0].transpose(0, 2, 1))
    # per prompt: the largest off-<start> score has code 0 and de-quantizes to exactly s
    for b in range(B):
        rest = A[b, :, :, 1:]
        h, i, j = np.unravel_index(np.argmax(rest), rest.shape)
        assert float(s[b].ravel()[0]) == rest[h, i, j]
        assert codes[b, h, i, j] == 0
        Vj = np.zeros_like(V, dtype=np.float64); Vj[:, j + 1] = 1.0
        Oj, *_ = oa.cross_attn_logq(Q, K, Vj, bits)
        assert Oj[b, i, h, 0] == rest[h, i, j]
    # un-clamped entries are within a factor sqrt(2) of the score
    s_full = np.broadcast_to(s, codes.shape[:-1] + (1,))
    A_hat = np.ldexp(s_full, -codes)
    ok = codes < 2 ** bits - 1
    ratio = (A_hat / A[..., 1:])[ok]
    assert ratio.min() >= 2 ** -0.5 * (1 - 1e-12) and ratio.max() <= 2 ** 0.5 * (1 + 1e-12)


def test_codes_invariant_to_row_logit_shift():
    Q, K, V = _inputs(seed=3)
    _, c0, _, _ = oa.cross_attn_logq(Q, K, V, 8)
    delta = np.random.default_rng(0).standard_normal(K.shape[-1]) * 0.25
    K2 = K.astype(np.float64) + delta            # adds q_i . delta to every logit of row i
    _, c1, _, _ = oa.cross_attn_logq(Q, K2, V, 8)
    assert (c0 != c1).mean() < 1e-3 and np.abs(c0 - c1).max() <= 1


def test_lossless_case_equals_textbook_attention():
    """Logits that are integer multiples of ln 2 make every off-<start> score an exact power of
    two times the scale: codes are exact and the output is plain softmax attention."""
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(4)
    B, H, nq, nk, d = 2, 2, 12, 7, 4
    Q = np.zeros((B, nq, H, d)); Q[..., 0] = math.sqrt(d) * math.log(2.0)
    K = np.zeros((B, nk, H, d)); K[..., 0] = rng.integers(-6, 1, (B, nk, 1))      # same keys in every head: equal row sums
    K[:, 1, :, 0] = 0                      # the off-<start> maximum
    K[:, 0, :, 0] = 3                      # a dominant <start> column
    V = rng.standard_normal((B, nk, H, d))
    O, codes, s, A = oa.cross_attn_logq(Q, K, V, 8)
    assert np.array_equal(codes, np.broadcast_to(-K[:, 1:, :, 0].transpose(0, 2, 1)[:, :, None, :], codes.shape))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q).permute(0, 2, 1, 3), torch.from_numpy(K).permute(0, 2, 1, 3),
        torch.from_numpy(V).permute(0, 2, 1, 3)).permute(0, 2, 1, 3).numpy()
    assert np.max(np.abs(O - ref)) < 1e-13


def test_scale_granularity_and_fixed_scale():
    Q, K, V = _inputs(seed=5)
    A = oa.softmax_scores(Q, K)
    sp = oa.prompt_scale(A, oa.PER_PROMPT)
    sh = oa.prompt_scale(A, oa.PER_PROMPT_HEAD)
    sc = oa.prompt_scale(A, oa.PER_CALL)
    assert np.array_equal(sp.ravel(), sh.max(axis=1).ravel())
    assert sc.ravel()[0] == sp.max()
    # static variant with the dynamic scale passed in reproduces the dynamic result
    O, codes, s, _ = oa.cross_attn_logq(Q, K, V, 8)
    O2, codes2, _, _ = oa.cross_attn_logq(Q, K, V, 8, fixed_scale=sp.ravel())
    assert np.array_equal(codes, codes2) and np.array_equal(O, O2)
    with pytest.raises(ValueError):
        oa.cross_attn_logq(Q, K[:, :1], V[:, :1], 8)


def test_four_bit_agrees_with_eight_bit_below_saturation():
    Q, K, V = _inputs(seed=6)
    _, c8, _, _ = oa.cross_attn_logq(Q, K, V, 8)
    _, c4, _, _ = oa.cross_attn_logq(Q, K, V, 4)
    assert np.array_equal(c4[c8 <= 15], c8[c8 <= 15]) and np.all(c4[c8 > 15] == 15)


# ---------------------------------------------------------------------------------------------- quantized V_hat
def test_quantized_values_error_bound_and_grid():
    """V_hat lies on the grid s (q - Z) of its head's slab and is within s / 2 (+ fp16 rounding) of V."""
    rng = np.random.default_rng(5)
    V = rng.normal(0, 1, (2, 9, 3, 8)).astype(np.float16)
    for bits in (8, 4):
        V_hat, codes, s, Z = oa.quantize_values(V, bits)
        assert codes.min() >= 0 and codes.max() <= 2 ** bits - 1
        span = V.astype(np.float64).max(axis=(1, 3)) - V.astype(np.float64).min(axis=(1, 3))
        assert np.allclose(s, span / 2 ** bits, rtol=1e-6)                     # Eq. 6 over the slab
        grid = s[:, None, :, None].astype(np.float64) * (codes - Z[:, None, :, None])
        assert np.array_equal(V_hat[:, 0], grid[:, 0].astype(np.float32).astype(np.float64))
        assert np.max(np.abs(V_hat[:, 1:] - grid[:, 1:])) <= 2.0 ** -10 * np.abs(grid).max()   # fp16 operand
        # interior values round to the nearest level; the top of the range clips by one more half level
        # (Eq. 6 divides by 2^b, so the maximum maps one level past the last code)
        err = np.abs(V_hat - V.astype(np.float64))
        bound = (1.5 * s[:, None, :, None] + 2.0 ** -10 * np.abs(V.astype(np.float64)).max())
        assert (err <= bound).all()
        inner = codes < 2 ** bits - 1
        assert (err[inner] <= (0.5 * s[:, None, :, None] * np.ones_like(err))[inner] * (1 + 1e-6)
                + 2.0 ** -10 * np.abs(V.astype(np.float64)).max()).all()


def test_quantized_values_are_a_fixed_point_on_two_levels():
    """A slab that holds only its minimum and the value one grid step below its maximum is reproduced."""
    V = np.zeros((1, 4, 1, 4), np.float16)
    V[0, 1:, 0, ::2] = 1.0                        # lo = 0, hi = 1 -> s = 2^-8, level 256 clips to 255
    V_hat, codes, s, Z = oa.quantize_values(V, 8)
    assert Z[0, 0] == 0 and s[0, 0] == np.float32(2.0 ** -8)
    assert set(np.unique(codes)) == {0, 255}
    assert np.array_equal(np.unique(V_hat), np.array([0.0, 255.0 / 256.0]))


def test_attention_with_quantized_values_is_eq9_on_v_hat():
    """cross_attn_logq(v_bits) equals Eq. 9 evaluated with V replaced by quantize_values(V); a wide V_hat
    grid (16 bits) leaves the output within the grid step of the unquantized-V result."""
    Q, K, V = synth.attention_inputs(6, 2, 2, 24, 9, 8, ctx_dim=16)
    O_q, codes, s, A = oa.cross_attn_logq(Q, K, V, 8, v_bits=4)
    V_hat = oa.quantize_values(V, 4)[0]
    assert np.array_equal(O_q, oa.split_product(A, codes, s, V_hat))
    O, _, _, _ = oa.cross_attn_logq(Q, K, V, 8)
    assert np.max(np.abs(O_q - O)) > 0                                        # 4-bit values do move the output
    step = oa.quantize_values(V, 4)[2].max()
    # every output is a combination of values with weights that sum to at most ~1 (+ top-level clip)
    assert np.max(np.abs(O_q - O)) <= 1.5 * step * 1.01 + 1e-3


# ---------------------------------------------------------------------------------------------- self-attention
def test_self_attention_uniform_scores_are_exact():
    """Q = 0: every score is 1 / n_k, the row maximum is the scale, every code is 0 and the output is the
    plain mean of V, exactly what unquantized attention gives."""
    rng = np.random.default_rng(11)
    B, nq, nk, H, d = 2, 5, 7, 3, 4
    Q = np.zeros((B, nq, H, d), np.float16)
    K = rng.normal(0, 1, (B, nk, H, d)).astype(np.float16)
    V = rng.normal(0, 1, (B, nk, H, d)).astype(np.float16)
    O, codes, s, A = oa.self_attn_logq(Q, K, V, 8)
    assert not codes.any()
    assert np.allclose(s, 1.0 / nk)
    assert np.allclose(O, np.broadcast_to(V.astype(np.float64).mean(axis=1)[:, None], O.shape), atol=1e-12)
    assert np.allclose(O, oa.attention_reference(Q, K, V), atol=1e-12)


def test_self_attention_log_levels_and_error_bound():
    """Eq. 2 with the row maximum as scale: the largest score of a row gets code 0 and is reproduced; every
    unclamped score is reproduced within a factor 2^(+-1/2); codes grow by one per halving of the score."""
    Q, K, V = synth.attention_inputs(12, 2, 2, 20, 33, 8, ctx_dim=16)
    O, codes, s, A = oa.self_attn_logq(Q, K, V, 8)
    imax = A.argmax(axis=-1)
    assert (np.take_along_axis(codes, imax[..., None], axis=-1) == 0).all()
    A_hat = s * np.exp2(-codes.astype(np.float64))
    assert np.allclose(np.take_along_axis(A_hat, imax[..., None], axis=-1), A.max(axis=-1, keepdims=True))
    free = codes < 255
    ratio = A_hat[free] / A[free]
    assert ratio.min() >= 2.0 ** -0.5 - 1e-12 and ratio.max() <= 2.0 ** 0.5 + 1e-12
    assert np.array_equal(codes, np.clip(np.rint(-np.log2(A / s)), 0, 255).astype(np.int64))
    assert np.array_equal(O, oa.self_product(codes, s, V))


def test_self_attention_fixed_scale_and_clamping():
    """A fixed scale of 1 (the largest value a softmax score can take) with 3 bits: scores below 2^-7.5 all
    take the last code; the output is the explicit sum over keys."""
    Q, K, V = synth.attention_inputs(13, 1, 1, 6, 40, 8, ctx_dim=16)
    O, codes, s, A = oa.self_attn_logq(Q, K, V, 3, fixed_scale=np.array([1.0]))
    assert codes.max() == 7 and (codes[A < 2.0 ** -7.5] == 7).all()
    want = np.zeros_like(O)
    for q in range(6):
        for k in range(40):
            want[0, q, 0] += 2.0 ** -int(codes[0, 0, q, k]) * V[0, k, 0].astype(np.float64)
    assert np.allclose(O, want, atol=1e-12)
