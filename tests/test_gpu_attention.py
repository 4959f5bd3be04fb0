"""GPU parity: cross-attention with log2-quantized scores against the fp64 oracle."""
import numpy as np
import pytest

from oracle import attention as oa
from paper_2501_04304_b200 import synth
from dgq_testlib import gpu, to_dev, check_output, check_codes, flipped_output_bound

pytestmark = pytest.mark.gpu


def _compare(torch, b, Q, K, V, bits, gran=0, fixed=None, out_rel=1e-3, v_bits=None):
    O_ref, codes_ref, s_ref, A = oa.cross_attn_logq(Q, K, V, bits, gran, fixed, v_bits=v_bits)
    fx = to_dev(torch, np.asarray(fixed, np.float32)) if fixed is not None else None
    O, scale, codes = b.cross_attn_logq(to_dev(torch, Q), to_dev(torch, K), to_dev(torch, V), bits, gran, fx,
                                        want_scale=True, want_codes=True, v_bits=v_bits or 0)
    if v_bits:
        V = oa.quantize_values(V, v_bits)[0]      # the value operand both sides multiply with
    assert b.device_status() == 0
    s_gpu = scale.cpu().numpy().astype(np.float64)
    assert np.allclose(s_gpu, s_ref.ravel(), rtol=2e-5, atol=0)
    c = codes.cpu().numpy().astype(np.int64)
    diff = check_codes(c, codes_ref)
    # A score that sits on a rounding boundary may take either neighbouring level (softmax rounding).
    # The output is held to the oracle's own output, every row, with the allowance that the row's
    # flipped codes (if any) explain and nothing more ...
    Og = O.float().cpu().numpy().astype(np.float64)
    bound = out_rel * np.max(np.abs(O_ref)) + flipped_output_bound(diff, c, codes_ref, s_ref, V[:, 1:])
    assert np.all(np.abs(Og - O_ref) <= bound), f"max excess {np.max(np.abs(Og - O_ref) - bound):.3e}"
    # ... and, tighter, to Eq. 9 evaluated with the codes the kernel chose.
    check_output(O, oa.split_product(A, c, s_ref, V), out_rel)
    return int((diff != 0).sum())


@pytest.mark.parametrize("bits", [8, 4])
def test_small_config3_like(bits):
    torch, b = gpu()
    Q, K, V = synth.attention_inputs(3, 2, 8, 300, 77, 40)
    _compare(torch, b, Q, K, V, bits)


@pytest.mark.parametrize("B,H,nq,nk,d", [
    (1, 1, 16, 3, 40),       # tiny: one warp slab, nk far below the padded width
    (2, 3, 130, 77, 80),     # ragged row block
    (1, 2, 64, 77, 160),
    (1, 2, 257, 100, 64),    # nk > 80 path
    (2, 2, 40, 128, 128),
    (3, 1, 129, 2, 40),      # smallest legal nk
])
def test_shapes(B, H, nq, nk, d):
    torch, b = gpu()
    Q, K, V = synth.attention_inputs(4, B, H, nq, nk, d, ctx_dim=64)
    _compare(torch, b, Q, K, V, 8)


@pytest.mark.parametrize("gran", [0, 2])
def test_grid_beyond_one_resident_wave(gran):
    """8 x 16 heads x 3 row blocks = 384 thread blocks do not fit the device at once (2 per SM), so the call
    cannot meet at a grid barrier and takes its two-kernel route; same checks as everywhere."""
    torch, b = gpu()
    Q, K, V = synth.attention_inputs(12, 8, 16, 768, 77, 40, ctx_dim=64)
    _compare(torch, b, Q, K, V, 8, gran=gran)


@pytest.mark.parametrize("gran", [0, 1, 2])
def test_scale_granularity(gran):
    torch, b = gpu()
    Q, K, V = synth.attention_inputs(5, 3, 4, 200, 77, 40, ctx_dim=64)
    _compare(torch, b, Q, K, V, 6, gran=gran)


def test_fixed_scale_variant():
    torch, b = gpu()
    Q, K, V = synth.attention_inputs(6, 2, 2, 128, 77, 40, ctx_dim=64)
    _compare(torch, b, Q, K, V, 8, fixed=[0.05, 0.01])


def test_wide_logits_saturate_four_bits():
    """Spread-out logits: 4-bit codes clamp at 15 and the 8-bit codes run far past the fp16 range."""
    torch, b = gpu()
    Q, K, V = synth.attention_inputs(7, 1, 2, 256, 77, 40, ctx_dim=64)
    K = (K.astype(np.float32) * 6).astype(np.float16)
    K[:, 0, :, -1] = np.float16(6.0 * np.sqrt(40))
    for bits in (4, 8):
        O_ref, codes_ref, _, _ = oa.cross_attn_logq(Q, K, V, bits)
        assert codes_ref.max() == (15 if bits == 4 else codes_ref.max()) and codes_ref.max() >= 15
        _compare(torch, b, Q, K, V, bits)


def test_uniform_and_one_hot_scores():
    """Degenerate softmax rows.  Q = 0 gives every key the score 1 / nk: the scale is 1 / nk, every code is 0
    and the output is the mean of V.  A <start> logit far above the rest leaves the other columns a total
    weight of about e^-60: the scale follows them down to about 2.5e-26, the codes stay small relative to it
    and the output is V[0]."""
    torch, b = gpu()
    Q, K, V = synth.attention_inputs(12, 2, 2, 200, 77, 40, ctx_dim=64)
    Q0 = np.zeros_like(Q)
    O_ref, codes_ref, s_ref, _ = oa.cross_attn_logq(Q0, K, V, 8)
    assert codes_ref.max() == 0 and np.allclose(s_ref, 1.0 / 77)
    assert np.allclose(O_ref, V.astype(np.float64).mean(axis=1)[:, None], rtol=0, atol=1e-12)
    _compare(torch, b, Q0, K, V, 8)
    K1 = K.copy()
    K1[:, 0, :, -1] = np.float16(60.0 * np.sqrt(40))      # the <start> column gets e^60 times the others' weight
    O_ref, codes_ref, _, _ = oa.cross_attn_logq(Q, K1, V, 4)
    assert np.allclose(O_ref, V[:, :1].astype(np.float64), rtol=0, atol=1e-6)
    _compare(torch, b, Q, K1, V, 4)
    _compare(torch, b, Q, K1, V, 8)


def test_argument_errors():
    torch, b = gpu()
    Q, K, V = synth.attention_inputs(8, 1, 1, 16, 4, 40, ctx_dim=16)
    Qd, Kd, Vd = to_dev(torch, Q), to_dev(torch, K), to_dev(torch, V)
    with pytest.raises(b.DgqError) as e:
        b.cross_attn_logq(Qd, Kd[:, :1].contiguous(), Vd[:, :1].contiguous())
    assert e.value.status == 1
    with pytest.raises(b.DgqError) as e:
        b.cross_attn_logq(Qd, Kd, Vd, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 4


@pytest.mark.parametrize("v_bits", [8, 6, 4])
def test_quantized_value_operand(v_bits):
    """Eq. 9 with V_hat: the kernel quantizes each head's value slab itself; the oracle's V_hat enters the
    comparison, so a wrong range, zero-point or code shows as an output error far above the tolerance."""
    torch, b = gpu()
    Q, K, V = synth.attention_inputs(8, 2, 4, 300, 77, 40)
    _compare(torch, b, Q, K, V, 8, v_bits=v_bits)


@pytest.mark.parametrize("B,H,nq,nk,d", [(1, 2, 64, 77, 160), (2, 2, 40, 128, 128), (3, 1, 129, 2, 40), (1, 3, 257, 100, 64)])
def test_quantized_value_operand_shapes(B, H, nq, nk, d):
    torch, b = gpu()
    Q, K, V = synth.attention_inputs(9, B, H, nq, nk, d, ctx_dim=64)
    _compare(torch, b, Q, K, V, 8, v_bits=8)


def test_quantized_value_operand_rejects_bad_bits():
    torch, b = gpu()
    Q, K, V = [to_dev(torch, x) for x in synth.attention_inputs(10, 1, 1, 16, 4, 40, ctx_dim=16)]
    for bad in (1, 9):
        with pytest.raises(Exception):
            b.cross_attn_logq(Q, K, V, 8, v_bits=bad)
