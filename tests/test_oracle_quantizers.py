"""Pins for the oracle's quantizer primitives (Eq. 1, Eq. 2, Eq. 6) and cost identities."""
import math
import os

import numpy as np
import pytest

from oracle import quantizers as oq
from oracle import cost

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_eq1_hand_example():
    # s = 0.5, z = 3, b = 4: x/s = -4, -2.6, 0, 1.48, 2.52, 20 -> round -> +3 -> clamp to [0, 15]
    x = [-2.0, -1.3, 0.0, 0.74, 1.26, 10.0]
    q = oq.linear_quantize(x, 0.5, 3, 4)
    assert q.tolist() == [0, 0, 3, 4, 6, 15]
    dq = oq.linear_dequantize(q, 0.5, 3)
    assert dq.tolist() == [-1.5, -1.5, 0.0, 0.5, 1.5, 6.0]


def test_eq1_half_to_even():
    # ties: 0.5 -> 0, 1.5 -> 2, 2.5 -> 2
    assert oq.linear_quantize([0.5, 1.5, 2.5], 1.0, 0, 8).tolist() == [0, 2, 2]


def test_eq2_hand_example():
    # x/s = 1, 1/2, 1/4, 0.3 (-log2 = 1.737 -> 2), 0.72 (0.474 -> 0), 2 (-1 -> clamp 0), 0 (inf -> L)
    s = 0.04
    x = [s, s / 2, s / 4, 0.3 * s, 0.72 * s, 2 * s, 0.0]
    assert oq.log_quantize(x, s, 4).tolist() == [0, 1, 2, 2, 0, 0, 15]
    assert oq.log_quantize([s * 2.0 ** -40], s, 8).tolist() == [40]
    assert oq.log_quantize([s * 2.0 ** -40], s, 4).tolist() == [15]


@pytest.mark.parametrize("b", [4, 6, 8])
def test_code_ranges(b):
    rng = np.random.default_rng(b)
    x = rng.standard_normal(5000) * 10
    lo, hi = x.min(), x.max()
    s, inv_s, Z = oq.group_params(lo, hi, b)
    q = oq.linear_quantize(x, s, Z, b)
    assert q.min() >= 0 and q.max() <= 2 ** b - 1
    qc = oq.quantize_canonical_f32(x, inv_s, Z, b)
    assert qc.min() >= 0 and qc.max() <= 2 ** b - 1
    p = np.abs(rng.standard_normal(5000)) * 1e-3
    ql = oq.log_quantize(p, p.max(), b)
    assert ql.min() == 0 and ql.max() <= 2 ** b - 1


@pytest.mark.parametrize("b", [4, 6, 8])
def test_linear_error_bounds_and_roundtrip(b):
    rng = np.random.default_rng(10 + b)
    x = rng.uniform(-3, 5, 20000)
    lo, hi = float(x.min()), float(x.max())
    s, inv_s, Z = oq.group_params(lo, hi, b)
    L = 2 ** b - 1
    q = oq.linear_quantize(x, s, Z, b)
    dq = oq.linear_dequantize(q, s, Z)
    s64 = float(s)
    inside = (x >= s64 * (0 - Z)) & (x <= s64 * (L - Z))
    assert np.all(np.abs(x - dq)[inside] <= s64 / 2 * (1 + 1e-9))
    # Eq. 6 divides by 2^b, so the top of the range clamps: hi - s (L - Z) = s + (lo + s Z),
    # and |lo + s Z| <= s / 2 by the rounding of Z
    assert np.all(np.abs(x - dq) <= 1.5 * s64 * (1 + 1e-6))
    # idempotence
    assert np.array_equal(oq.linear_quantize(dq, s, Z, b), q)
    # monotone
    xs = np.sort(x)
    assert np.all(np.diff(oq.linear_quantize(xs, s, Z, b)) >= 0)
    # zero maps to the zero-point and back to exactly zero
    assert 0 <= Z <= L
    assert oq.linear_quantize([0.0], s, Z, b)[0] == Z
    assert oq.linear_dequantize([Z], s, Z)[0] == 0.0
    # minimum maps to code 0, maximum to the last code
    assert q[np.argmin(x)] == 0 and q[np.argmax(x)] == L


def test_group_params_literal_denominator():
    s, inv_s, Z = oq.group_params(-1.0, 3.0, 8)
    assert float(s) == 4.0 / 256.0            # 2^b, not 2^b - 1
    assert float(inv_s) == 64.0
    assert Z == 64
    s, _, Z = oq.group_params(2.0, 2.0, 8)     # constant group
    assert float(s) == float(np.float32(1e-8))
    s, _, Z = oq.group_params(1.0, 3.0, 4)     # all-positive group: negative zero-point
    assert Z == -8


def test_canonical_f32_close_to_ideal():
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(200000) * 3).astype(np.float16).astype(np.float32)
    s, inv_s, Z = oq.group_params(x.min(), x.max(), 8)
    qc = oq.quantize_canonical_f32(x, inv_s, Z, 8)
    qi = oq.linear_quantize(x.astype(np.float64), float(s), Z, 8)
    diff = np.abs(qc - qi)
    assert diff.max() <= 1
    assert (diff != 0).mean() < 1e-3


def test_canonical_f32_nonfinite():
    x = np.array([np.nan, np.inf, -np.inf], dtype=np.float32)
    assert oq.quantize_canonical_f32(x, np.float32(4.0), 10, 8).tolist() == [0, 255, 0]


def test_log_levels_are_powers_of_two():
    rng = np.random.default_rng(2)
    p = rng.uniform(1e-9, 1.0, 10000)
    s = p.max()
    for b in (4, 6, 8):
        q = oq.log_quantize(p, s, b)
        dq = oq.log_dequantize(q, s)
        mant, _ = np.frexp(dq / s)
        assert np.all(mant == 0.5)                        # exact powers of two
        assert q[np.argmax(p)] == 0 and dq[np.argmax(p)] == s
        unclamped = q < 2 ** b - 1
        ratio = dq[unclamped] / p[unclamped]
        assert np.all(ratio >= 2 ** -0.5 * (1 - 1e-12)) and np.all(ratio <= 2 ** 0.5 * (1 + 1e-12))
    q8 = oq.log_quantize(p, s, 8)
    q4 = oq.log_quantize(p, s, 4)
    assert np.array_equal(q4[q8 <= 15], q8[q8 <= 15])
    assert np.all(q4[q8 > 15] == 15)


def test_table2_bops_follow_from_identity():
    rows = [l.split() for l in open(os.path.join(GOLD, "table2_bops.txt")) if not l.startswith("#")]
    fp = {m: float(v) for m, bw, ba, v in rows if bw == "32"}
    for m, bw, ba, v in rows:
        flops_T = fp[m] / (32 * 32)
        got = cost.bops(flops_T, int(bw), int(ba))
        digits = len(v.split(".")[1]) if "." in v else 0
        assert abs(got - float(v)) <= 0.5 * 10 ** -digits + 1e-9, (m, bw, ba, got, v)


def test_param_memory_figure():
    T, groups, factor, mb = open(os.path.join(GOLD, "param_memory.txt")).readlines()[1].split()
    # the printed 2.29 MB is reached when both the scale and the zero-point set are counted
    total = cost.table_bytes(int(T), int(groups), int(factor), 2)
    assert abs(total / 2 ** 20 - float(mb)) < 0.01
