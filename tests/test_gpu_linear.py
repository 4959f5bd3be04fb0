"""GPU parity: the group-quantized linear / conv layer against the oracle (int64 accumulate, fp64 de-quantize)."""
import numpy as np
import pytest

from oracle import calibration as oc
from oracle import linear as ol
from paper_2501_04304_b200 import synth
from dgq_testlib import gpu, to_dev, unpermute_codes, layer_case, check_output

pytestmark = pytest.mark.gpu

REL = 1e-3   # max|delta| <= 1e-3 * max|ref|


def _run_linear(torch, b, X, W, bias, gr, g, mode, w_bits):
    wq_ref, sw_ref = ol.weight_rtn(W, w_bits)
    w = b.weight_prepare(g, to_dev(torch, W), w_bits)
    wq, sw = w.export()
    assert np.array_equal(wq, wq_ref) and np.array_equal(sw, sw_ref)
    Xd = to_dev(torch, X)
    bd = to_dev(torch, bias) if bias is not None else None
    if mode == "static":
        codes, s_rows, z_rows = ol.quantize_static(X, gr, 0)
        Xq, ds, dz = b.quantize_act(g, Xd)
        Y = b.linear(g, w, Xq, bias=bd)
    else:
        codes, s_rows, z_rows = ol.quantize_dynamic_token(X, gr.col_group, gr.G, gr.bits)
        Xq, ds, dz = b.quantize_act(g, Xd, mode=b.MODE_DYNAMIC_TOKEN)
        Y = b.linear(g, w, Xq, mode=b.MODE_DYNAMIC_TOKEN, dyn_scale=ds, dyn_zp=dz, bias=bd)
    assert np.array_equal(unpermute_codes(Xq, g.export()["perm"], X.shape[1]), codes)
    Yref = ol.group_linear(codes, s_rows, z_rows, gr.col_group, wq_ref, sw_ref, bias)
    assert b.device_status() == 0
    return check_output(Y, Yref, REL)


@pytest.mark.parametrize("mode", ["static", "dynamic"])
def test_config1_w8a8(mode):
    """256 tokens x 320 channels, 4 channel groups + outlier group, both outlier types, W8A8."""
    torch, b = gpu()
    Xcal, X, W, bias, gr = layer_case(0, 1, 256, 320, 320, 4, 8, oc.DIM_BOTH, oc.OUTLIER_EXPLICIT, 4, 2)
    g = b.calibrate_groups(to_dev(torch, Xcal), 256, 8, 4, b.DIM_BOTH, b.OUTLIER_EXPLICIT, 5.0)
    assert g.G == 5
    _run_linear(torch, b, X, W, bias, gr, g, mode, 8)


@pytest.mark.parametrize("M,C,N,K,w_bits,mode", [
    (128, 32, 16, 1, 8, "static"),          # one tile, one atom, one group
    (128, 32, 16, 1, 4, "static"),
    (1000, 320, 320, 8, 8, "dynamic"),      # ragged M tail, BN = 160
    (1000, 320, 320, 8, 4, "dynamic"),
    (616, 768, 640, 8, 4, "dynamic"),       # cross-attention k/v projection shape, M = 8 x 77
    (384, 1280, 320, 8, 8, "static"),       # FF2-like: long K, several stages per group
    (300, 320, 2560, 8, 8, "dynamic"),      # FF1-like: many N tiles
    (260, 328, 72, 16, 8, "dynamic"),       # N not a tile multiple (BN = 128 with tail), G = 16
    (130, 64, 48, 3, 4, "static"),          # BN = 64 path
])
def test_linear_shapes(M, C, N, K, w_bits, mode):
    torch, b = gpu()
    Xcal, X, W, bias, gr = layer_case(7, 1, M, C, N, K, 8, oc.DIM_CHANNEL)
    g = b.calibrate_groups(to_dev(torch, Xcal), M, 8, K, b.DIM_CHANNEL)
    _run_linear(torch, b, X, W, bias, gr, g, mode, w_bits)


def test_static_grid_with_pixel_groups_and_no_bias():
    torch, b = gpu()
    Xcal, X, W, bias, gr = layer_case(8, 2, 256, 320, 320, 4, 8, oc.DIM_BOTH)
    g = b.calibrate_groups(to_dev(torch, Xcal), 256, 8, 4, b.DIM_BOTH)
    assert g.R > 1 and g.G > 1
    _run_linear(torch, b, X, W, None, gr, g, "static", 8)


def test_a6_codes_and_centred_linear():
    """6-bit activations; zero-centred signed codes give the same layer output with no zero-point term."""
    torch, b = gpu()
    Xcal, X, W, bias, gr = layer_case(9, 1, 512, 320, 320, 8, 6, oc.DIM_CHANNEL, token_outliers=False)
    g = b.calibrate_groups(to_dev(torch, Xcal), 512, 6, 8, b.DIM_CHANNEL)
    wq, sw = ol.weight_rtn(W, 4)
    w = b.weight_prepare(g, to_dev(torch, W), 4)
    codes, s_rows, z_rows = ol.quantize_static(X, gr, 0)
    Yref = ol.group_linear(codes, s_rows, z_rows, gr.col_group, wq, sw, bias)
    Xd, bd = to_dev(torch, X), to_dev(torch, bias)
    Xq, _, _ = b.quantize_act(g, Xd, layout=b.CODES_S8_CENTRED)
    Y = b.linear(g, w, Xq, layout=b.CODES_S8_CENTRED, bias=bd)
    check_output(Y, Yref, REL)
    Xq2, _, _ = b.quantize_act(g, Xd)
    Y2 = b.linear(g, w, Xq2, bias=bd)
    check_output(Y2, Yref, REL)
    assert b.device_status() == 0


@pytest.mark.parametrize("n,H,W,C,N,K", [
    (2, 8, 8, 64, 64, 4),        # two images per row tile
    (1, 16, 16, 96, 160, 8),     # 8 image rows per tile
    (2, 32, 32, 320, 320, 16),   # 4 image rows per tile, G = 16
    (1, 64, 64, 64, 128, 3),     # 2 image rows per tile
])
def test_conv3x3_w4a6(n, H, W, C, N, K):
    torch, b = gpu()
    P = H * W
    Xcal = synth.activations(11, 100, 2 * n, P, C, None, None, token_outliers=False)
    X = synth.activations(11, 1, n, P, C, None, None, token_outliers=False)
    Wt = synth.conv_weights(11, 2, N, C)
    bias = synth.bias(11, 3, N)
    gr = oc.calibrate(Xcal, P, 6, K, dim_select=oc.DIM_CHANNEL)
    g = b.calibrate_groups(to_dev(torch, Xcal), P, 6, K, b.DIM_CHANNEL)
    wq, sw = ol.weight_rtn(Wt, 4)
    codes, s_rows, z_rows = ol.quantize_static(X, gr, 0)
    Yref = ol.group_conv3x3(codes.reshape(n, H, W, C), gr.scale[0][0], gr.zp[0][0], gr.col_group, wq, sw, bias)
    conv = (n, H, W, C)
    w = b.weight_prepare(g, to_dev(torch, Wt), 4, conv=conv)
    Xq, _, _ = b.quantize_act(g, to_dev(torch, X), layout=b.CODES_S8_CENTRED)
    Y = b.linear(g, w, Xq, layout=b.CODES_S8_CENTRED, bias=to_dev(torch, bias), conv=conv)
    assert b.device_status() == 0
    check_output(Y, Yref.reshape(n * P, N), REL)


def test_linear_argument_errors():
    torch, b = gpu()
    Xcal, X, W, bias, gr = layer_case(12, 1, 128, 64, 64, 2, 8, oc.DIM_CHANNEL)
    g = b.calibrate_groups(to_dev(torch, Xcal), 128, 8, 2, b.DIM_CHANNEL)
    w = b.weight_prepare(g, to_dev(torch, W), 8)
    Xq, _, _ = b.quantize_act(g, to_dev(torch, X))
    with pytest.raises(b.DgqError) as e:          # dynamic mode without its parameter arrays
        b.linear(g, w, Xq, mode=b.MODE_DYNAMIC_TOKEN)
    assert e.value.status == 1
    with pytest.raises(b.DgqError) as e:          # conv descriptor on a linear weight
        b.linear(g, w, Xq, conv=(1, 8, 16, 64))
    assert e.value.status == 1
    Y = torch.empty((128, 72), dtype=torch.float16, device="cuda")[:, 4:68]
    with pytest.raises(b.DgqError) as e:          # output not 16-byte aligned
        b.linear(g, w, Xq, out=Y)
    assert e.value.status == 2


@pytest.mark.parametrize("w_bits", [8, 4])
def test_objects_rebuilt_from_exports_give_identical_results(w_bits):
    """dgq_groups_export -> dgq_groups_from_host and dgq_weight_export -> dgq_weight_from_codes: the rebuilt
    grouping has the same layout and tables, the rebuilt weight the same codes, and the layer output is bit for
    bit the same (static grid with pixel and channel groups)."""
    torch, b = gpu()
    P, C, N, K = 256, 320, 320, 4
    Xcal, X, W, bias, gr = layer_case(14, 2, P, C, N, K, 8, oc.DIM_BOTH)
    g = b.calibrate_groups(to_dev(torch, Xcal), P, 8, K, b.DIM_BOTH)
    ex = g.export()
    g2 = b.groups_from_host(C, P, 8, ex["col_group"], ex["row_group"], ex["scale"], ex["zp"])
    ex2 = g2.export()
    assert (g2.G, g2.R, g2.T, g2.K_pad, g2.bits) == (g.G, g.R, g.T, g.K_pad, g.bits)
    for k in ("perm", "col_group", "group_off", "row_group", "scale", "zp"):
        assert np.array_equal(ex[k], ex2[k]), k
    w = b.weight_prepare(g, to_dev(torch, W), w_bits)
    wq, sw = w.export()
    w2 = b.weight_from_codes(g2, wq, sw, w_bits)
    wq2, sw2 = w2.export()
    assert np.array_equal(wq, wq2) and np.array_equal(sw, sw2)
    Xd, bd = to_dev(torch, X), to_dev(torch, bias)
    Xq, _, _ = b.quantize_act(g, Xd)
    Xq2, _, _ = b.quantize_act(g2, Xd)
    assert torch.equal(Xq, Xq2)
    Y = b.linear(g, w, Xq, bias=bd)
    Y2 = b.linear(g2, w2, Xq2, bias=bd)
    assert torch.equal(Y, Y2)
    codes, s_rows, z_rows = ol.quantize_static(X, gr, 0)
    check_output(Y2, ol.group_linear(codes, s_rows, z_rows, gr.col_group, *ol.weight_rtn(W, w_bits), bias), REL)
    assert b.device_status() == 0


def test_four_bit_weights_with_and_without_workspace():
    """4-bit weights take two routes: expanded once per call into the caller's workspace in front of the GEMM, or,
    without a workspace, expanded stage by stage inside it.  Same integers either way: identical outputs."""
    torch, b = gpu()
    M, C, N, K = 1000, 640, 640, 8
    Xcal, X, W, bias, gr = layer_case(15, 1, M, C, N, K, 8, oc.DIM_CHANNEL)
    g = b.calibrate_groups(to_dev(torch, Xcal), M, 8, K, b.DIM_CHANNEL)
    w = b.weight_prepare(g, to_dev(torch, W), 4)
    need = b.linear_workspace_bytes(g, w, M)
    assert need > 0
    Xq, ds, dz = b.quantize_act(g, to_dev(torch, X), mode=b.MODE_DYNAMIC_TOKEN)
    kw = dict(mode=b.MODE_DYNAMIC_TOKEN, dyn_scale=ds, dyn_zp=dz, bias=to_dev(torch, bias))
    Y_ws = b.linear(g, w, Xq, workspace=torch.empty(need, dtype=torch.uint8, device="cuda"), **kw)
    Y_in = b.linear(g, w, Xq, workspace=False, **kw)
    assert torch.equal(Y_ws, Y_in)
    with pytest.raises(b.DgqError) as e:          # a workspace that is too small is refused
        b.linear(g, w, Xq, workspace=torch.empty(need // 2, dtype=torch.uint8, device="cuda"), **kw)
    assert e.value.status == 4
    codes, s_rows, z_rows = ol.quantize_dynamic_token(X, gr.col_group, gr.G, gr.bits)
    check_output(Y_ws, ol.group_linear(codes, s_rows, z_rows, gr.col_group, *ol.weight_rtn(W, 4), bias), REL)
    assert b.device_status() == 0


def test_a_wait_that_runs_out_is_reported_and_leaves_the_device_usable():
    """Every device-side wait is bounded.  The library's self-test kernel waits, with a short limit, on a barrier
    nobody arrives at: the status word reads DGQ_ERR_TIMEOUT once, is clear afterwards, and a layer call right
    after it gives the right result."""
    torch, b = gpu()
    assert b.device_status() == 0
    b.selftest_wait_timeout(2000)
    assert b.device_status() == 6
    assert b.device_status() == 0
    Xcal, X, W, bias, gr = layer_case(16, 1, 256, 320, 320, 4, 8, oc.DIM_CHANNEL)
    g = b.calibrate_groups(to_dev(torch, Xcal), 256, 8, 4, b.DIM_CHANNEL)
    _run_linear(torch, b, X, W, bias, gr, g, "dynamic", 8)
