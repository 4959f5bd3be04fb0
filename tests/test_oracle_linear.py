"""Pins for the oracle's group-quantized linear / conv layer."""
import numpy as np
import pytest

from oracle import calibration as oc
from oracle import linear as ol
from oracle import quantizers as oq
from paper_2501_04304_b200 import synth


def test_int4_pack_roundtrip_all_bytes():
    allb = np.arange(256, dtype=np.uint8).reshape(256, 1)
    un = ol.unpack_int4(allb)
    assert un.min() == -8 and un.max() == 7
    assert np.array_equal(ol.pack_int4(un), allb)
    # low nibble is the even index, two's complement: 0xF1 -> (1, -1)
    assert ol.unpack_int4(np.array([[0xF1]], dtype=np.uint8)).tolist() == [[1, -1]]
    assert ol.unpack_int4(np.array([[0x8F]], dtype=np.uint8)).tolist() == [[-1, -8]]


@pytest.mark.parametrize("bits", [8, 4])
def test_weight_rtn_bounds(bits):
    W = synth.weights(1, 3, 40, 64)
    wq, sw = ol.weight_rtn(W, bits)
    qmax = 2 ** (bits - 1) - 1
    assert wq.min() >= -qmax and wq.max() <= qmax
    err = np.abs(W.astype(np.float64) - sw.astype(np.float64)[:, None] * wq)
    assert np.all(err <= sw.astype(np.float64)[:, None] / 2 * (1 + 1e-5))
    # the row's largest magnitude sits on the last code
    assert np.all(np.abs(wq).max(axis=1) == qmax)
    wz, sz = ol.weight_rtn(np.zeros((2, 8), np.float16), bits)
    assert np.all(wz == 0) and np.all(sz == 1.0)


def _setup(seed=0, M=48, P=16, C=40, N=24, K=3, bits=8, wbits=8, dim=oc.DIM_BOTH):
    Xcal = synth.activations(seed, 100, 4, P, C, n_out_ch=2, n_out_tok=1)
    X = synth.activations(seed, 1, M // P, P, C, n_out_ch=2, n_out_tok=1)
    W = synth.weights(seed, 2, N, C)
    b = synth.bias(seed, 3, N)
    gr = oc.calibrate(Xcal, P, bits, K, dim_select=dim)
    wq, sw = ol.weight_rtn(W, wbits)
    return X, W, b, gr, wq, sw


@pytest.mark.parametrize("mode", ["static", "dynamic"])
def test_zero_point_algebra_equals_fake_quant(mode):
    X, W, b, gr, wq, sw = _setup()
    if mode == "static":
        codes, s, z = ol.quantize_static(X, gr, 0)
    else:
        codes, s, z = ol.quantize_dynamic_token(X, gr.col_group, gr.G, 8)
    Y = ol.group_linear(codes, s, z, gr.col_group, wq, sw, b)
    Yf = ol.fake_quant_reference(codes, s, z, gr.col_group, wq, sw, b)
    assert np.max(np.abs(Y - Yf)) <= 1e-11 * np.max(np.abs(Yf))


def test_brute_force_tiny():
    """Every term of the layer formula written as scalar loops over de-quantized operands."""
    X, W, b, gr, wq, sw = _setup(seed=1, M=8, P=4, C=6, N=3, K=2)
    codes, s, z = ol.quantize_static(X, gr, 0)
    Y = ol.group_linear(codes, s, z, gr.col_group, wq, sw, b)
    for t in range(8):
        r = gr.row_group[t % 4]
        for o in range(3):
            acc = 0.0
            for c in range(6):
                g = gr.col_group[c]
                xdq = float(gr.scale[0][r, g]) * (int(codes[t, c]) - int(gr.zp[0][r, g]))
                acc += xdq * (float(sw[o]) * int(wq[o, c]))
            acc += float(b[o])
            assert abs(Y[t, o] - acc) <= 1e-12 * max(1.0, abs(acc))


def test_permutation_invariance():
    X, W, b, gr, wq, sw = _setup(seed=2)
    codes, s, z = ol.quantize_static(X, gr, 0)
    Y = ol.group_linear(codes, s, z, gr.col_group, wq, sw, b)
    perm = np.random.default_rng(0).permutation(X.shape[1])
    Yp = ol.group_linear(codes[:, perm], s, z, gr.col_group[perm], wq[:, perm], sw, b)
    assert np.array_equal(Y, Yp)


def test_high_precision_limit_is_plain_matmul():
    """With 16-bit codes on both operands the only error source (quantization) vanishes."""
    X, W, b, gr, _, _ = _setup(seed=3)
    codes, s, z = ol.quantize_dynamic_token(X, gr.col_group, gr.G, 16)
    wq16, sw16 = None, None
    Wf = W.astype(np.float32)
    qmax = np.float32(2 ** 15 - 1)
    sw16 = (np.abs(Wf).max(axis=1) / qmax).astype(np.float32)
    wq16 = np.rint(Wf / sw16[:, None]).astype(np.int64)
    Y = ol.group_linear(codes, s, z, gr.col_group, wq16, sw16, b)
    ref = X.astype(np.float64) @ W.astype(np.float64).T + b.astype(np.float64)
    assert np.max(np.abs(Y - ref)) <= 2e-4 * np.max(np.abs(ref))


def test_one_group_is_textbook_int8_gemm():
    X, W, b, _, wq, sw = _setup(seed=4)
    Xcal = synth.activations(4, 100, 4, 16, 40, n_out_ch=2, n_out_tok=1)
    gr = oc.calibrate(Xcal, 16, 8, 1, dim_select=oc.DIM_CHANNEL)
    codes, s, z = ol.quantize_static(X, gr, 0)
    Y = ol.group_linear(codes, s, z, gr.col_group, wq, sw, b)
    s0, z0 = float(gr.scale[0][0, 0]), int(gr.zp[0][0, 0])
    ref = s0 * ((codes.astype(np.int64) - z0) @ wq.astype(np.int64).T) * sw.astype(np.float64)[None, :] + b.astype(np.float64)
    assert np.max(np.abs(Y - ref)) <= 1e-12 * np.max(np.abs(ref))


def test_dynamic_token_hits_both_ends():
    X, _, _, gr, _, _ = _setup(seed=5)
    codes, s, z = ol.quantize_dynamic_token(X, gr.col_group, gr.G, 8)
    Xf = X.astype(np.float32)
    for g in range(gr.G):
        cols = np.flatnonzero(gr.col_group == g)
        if cols.size < 2:
            continue
        sub, q = Xf[:, cols], codes[:, cols]
        rows = np.arange(X.shape[0])
        assert np.all(q[rows, sub.argmin(axis=1)] == 0)
        assert np.all(q[rows, sub.argmax(axis=1)] == 255)
        assert np.allclose(s[:, g], (sub.max(1) - sub.min(1)) / 256.0)


def _conv_setup(seed=0, n=2, H=5, W=4, C=12, N=6, K=3, bits=6):
    Xcal = synth.activations(seed, 100, 2 * n, H * W, C, n_out_ch=1, token_outliers=False)
    X = synth.activations(seed, 1, n, H * W, C, n_out_ch=1, token_outliers=False)
    Wt = synth.conv_weights(seed, 2, N, C)
    b = synth.bias(seed, 3, N)
    gr = oc.calibrate(Xcal, H * W, bits, K, dim_select=oc.DIM_CHANNEL)
    wq, sw = ol.weight_rtn(Wt, 4)
    codes, s, z = ol.quantize_static(X, gr, 0)
    return X, Wt, b, gr, wq, sw, codes.reshape(n, H, W, C)


def test_conv_brute_force_seven_loops():
    X, Wt, b, gr, wq, sw, codes = _conv_setup()
    n, H, W, C = codes.shape
    s_g, z_g = gr.scale[0][0], gr.zp[0][0]
    Y = ol.group_conv3x3(codes, s_g, z_g, gr.col_group, wq, sw, b)
    for i in range(n):
        for h in range(H):
            for w in range(W):
                for o in range(wq.shape[0]):
                    acc = 0.0
                    for ky in range(3):
                        for kx in range(3):
                            hh, ww = h + ky - 1, w + kx - 1
                            if not (0 <= hh < H and 0 <= ww < W):
                                continue                      # zero padding of the de-quantized input
                            for c in range(C):
                                g = gr.col_group[c]
                                xdq = float(s_g[g]) * (int(codes[i, hh, ww, c]) - int(z_g[g]))
                                acc += xdq * float(sw[o]) * int(wq[o, ky, kx, c])
                    acc += float(b[o])
                    assert abs(Y[i, h, w, o] - acc) <= 1e-11 * max(1.0, abs(acc))


def test_conv_matches_library_correlation():
    scipy_signal = pytest.importorskip("scipy.signal")
    X, Wt, b, gr, wq, sw, codes = _conv_setup(seed=1, n=1, H=7, W=6, C=8, N=3)
    s_g, z_g = gr.scale[0][0], gr.zp[0][0]
    Y = ol.group_conv3x3(codes, s_g, z_g, gr.col_group, wq, sw, b)
    cg = gr.col_group
    Xdq = s_g.astype(np.float64)[cg] * (codes[0].astype(np.float64) - z_g.astype(np.float64)[cg])   # [H, W, C]
    for o in range(3):
        ref = np.zeros(Xdq.shape[:2])
        for c in range(8):
            ker = float(sw[o]) * wq[o, :, :, c].astype(np.float64)
            ref += scipy_signal.correlate2d(Xdq[:, :, c], ker, mode="same", boundary="fill", fillvalue=0.0)
        ref += float(b[o])
        assert np.max(np.abs(Y[0, :, :, o] - ref)) <= 1e-11 * max(1.0, np.max(np.abs(ref)))
