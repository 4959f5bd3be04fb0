"""GPU parity: attention with log2-quantized scores over all keys (self-attention) against the fp64 oracle."""
import numpy as np
import pytest

from oracle import attention as oa
from paper_2501_04304_b200 import synth
from dgq_testlib import gpu, to_dev, check_output, check_codes, flipped_output_bound

pytestmark = pytest.mark.gpu


def _compare(torch, b, Q, K, V, bits, fixed=None, out_rel=1e-3):
    O_ref, codes_ref, s_ref, A = oa.self_attn_logq(Q, K, V, bits, fixed)
    fx = to_dev(torch, np.asarray(fixed, np.float32)) if fixed is not None else None
    O, codes = b.self_attn_logq(to_dev(torch, Q), to_dev(torch, K), to_dev(torch, V), bits, fx, want_codes=True)
    torch.cuda.synchronize()
    assert b.device_status() == 0
    c = codes.cpu().numpy().astype(np.int64)
    diff = check_codes(c, codes_ref)
    # a score on a rounding boundary may take either neighbouring level: every row is held to the oracle's
    # output with the allowance its flipped codes (if any) explain, and to the product evaluated with the
    # codes the kernel chose
    Og = O.float().cpu().numpy().astype(np.float64)
    bound = out_rel * np.max(np.abs(O_ref)) + flipped_output_bound(diff, c, codes_ref, s_ref, V)
    assert np.all(np.abs(Og - O_ref) <= bound), f"max excess {np.max(np.abs(Og - O_ref) - bound):.3e}"
    check_output(O, oa.self_product(c, s_ref, V), out_rel)
    # the variant that writes no codes gives the same output
    O2, _ = b.self_attn_logq(to_dev(torch, Q), to_dev(torch, K), to_dev(torch, V), bits, fx)
    assert torch.equal(O, O2)


def _qkv(seed, B, H, n, d, nk=None):
    """Self-attention inputs: queries, keys and values of the same n tokens (seeded normal fp16)."""
    rng = np.random.default_rng((seed, 77))
    nk = n if nk is None else nk
    Q = rng.normal(0, 1, (B, n, H, d)).astype(np.float16)
    K = rng.normal(0, 1, (B, nk, H, d)).astype(np.float16)
    V = rng.normal(0, 1, (B, nk, H, d)).astype(np.float16)
    return Q, K, V


@pytest.mark.parametrize("bits", [8, 4])
def test_small_self_attention(bits):
    torch, b = gpu()
    Q, K, V = _qkv(1, 2, 3, 300, 40)          # 5 key blocks, ragged last block, ragged row block
    _compare(torch, b, Q, K, V, bits)


@pytest.mark.parametrize("B,H,n,nk,d", [
    (1, 1, 16, 3, 40),        # one partial key block
    (2, 2, 64, 64, 64),       # exactly one key block
    (1, 2, 130, 257, 80),     # nk != nq, ragged everything
    (1, 1, 129, 128, 128),
    (1, 2, 70, 65, 160),
])
def test_shapes(B, H, n, nk, d):
    torch, b = gpu()
    Q, K, V = _qkv(2, B, H, n, d, nk)
    _compare(torch, b, Q, K, V, 8)


def test_fixed_scale():
    torch, b = gpu()
    Q, K, V = _qkv(3, 2, 2, 200, 40)
    _compare(torch, b, Q, K, V, 6, fixed=[1.0, 0.25])


def test_level_at_1024_tokens():
    """32 x 32 level: 1024 tokens, 8 heads of 80 features; the whole output against the oracle."""
    torch, b = gpu()
    Q, K, V = _qkv(4, 1, 8, 1024, 80)
    _compare(torch, b, Q, K, V, 8)


def test_argument_errors():
    torch, b = gpu()
    Q, K, V = [to_dev(torch, x) for x in _qkv(5, 1, 1, 16, 40)]
    with pytest.raises(Exception):
        b.self_attn_logq(Q, K, V, 9)
    Q48 = torch.zeros((1, 16, 1, 48), dtype=torch.float16, device="cuda")
    with pytest.raises(Exception):
        b.self_attn_logq(Q48, Q48, Q48, 8)
