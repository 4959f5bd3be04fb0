"""GPU parity: calibration (grouping, tables) and the activation quantizer, bit-exact against the oracle."""
import numpy as np
import pytest

from oracle import calibration as oc
from oracle import linear as ol
from oracle.quantizers import quantize_canonical_f32
from paper_2501_04304_b200 import synth
from dgq_testlib import gpu, to_dev, unpermute_codes, oracle_grouping_matches, layer_case

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dim,mode,K", [
    (oc.DIM_AUTO, oc.OUTLIER_KMEANS, 8),
    (oc.DIM_CHANNEL, oc.OUTLIER_KMEANS, 16),
    (oc.DIM_PIXEL, oc.OUTLIER_KMEANS, 4),
    (oc.DIM_BOTH, oc.OUTLIER_EXPLICIT, 4),
])
def test_calibration_matches_oracle(dim, mode, K):
    torch, b = gpu()
    Xcal, X, W, bias, gr = layer_case(0, 1, 256, 320, 320, K, 8, dim, mode, n_out_ch=4, n_out_tok=2)
    g = b.calibrate_groups(to_dev(torch, Xcal), 256, 8, K, dim, mode, 5.0)
    assert (g.G, g.R, g.dim) == (gr.G, gr.R, gr.dim)
    assert abs(g.D_channel - gr.D_channel) < 1e-9 and abs(g.D_pixel - gr.D_pixel) < 1e-9
    ex = g.export()
    oracle_grouping_matches(gr, ex)
    # layout: every group padded to a multiple of 32, members in ascending channel order
    assert g.K_pad % 32 == 0 and np.all(ex["group_off"] % 32 == 0)
    for k in range(g.G):
        seg = ex["perm"][ex["group_off"][k]:ex["group_off"][k + 1]]
        mem = seg[seg >= 0]
        assert np.array_equal(mem, np.flatnonzero(gr.col_group == k))
    assert b.device_status() == 0


def test_calibration_timestep_rows():
    torch, b = gpu()
    X0 = synth.activations(5, 1, 2, 64, 64, n_out_ch=1, n_out_tok=1)
    X1 = (synth.activations(5, 2, 2, 64, 64, n_out_ch=1, n_out_tok=1).astype(np.float32) * 2).astype(np.float16)
    gr = oc.calibrate(X0, 64, 6, 3, dim_select=oc.DIM_BOTH, timestep=0)
    oc.fill_timestep(gr, X1, 2)
    g = b.calibrate_groups(to_dev(torch, X0), 64, 6, 3, b.DIM_BOTH, n_timesteps=3, timestep=0)
    b.calibrate_groups(to_dev(torch, X1), 64, 6, 3, b.DIM_BOTH, n_timesteps=3, timestep=2, groups=g)
    oracle_grouping_matches(gr, g.export())
    # the row that was never filled is refused
    with pytest.raises(b.DgqError) as e:
        b.quantize_act(g, to_dev(torch, X0), timestep=1)
    assert e.value.status == 7


@pytest.mark.parametrize("case", [
    dict(n=1, P=256, C=320, K=4, bits=8, dim=oc.DIM_BOTH, om=oc.OUTLIER_EXPLICIT, oc_=4, ot=2),   # config 1
    dict(n=3, P=100, C=328, K=8, bits=8, dim=oc.DIM_CHANNEL, om=oc.OUTLIER_KMEANS, oc_=None, ot=None),
    dict(n=2, P=77, C=768, K=16, bits=6, dim=oc.DIM_AUTO, om=oc.OUTLIER_KMEANS, oc_=None, ot=None),
    dict(n=1, P=33, C=2560, K=8, bits=8, dim=oc.DIM_PIXEL, om=oc.OUTLIER_KMEANS, oc_=None, ot=None),
    dict(n=1, P=5, C=8, K=2, bits=4, dim=oc.DIM_CHANNEL, om=oc.OUTLIER_KMEANS, oc_=1, ot=1),
])
def test_static_codes_bit_exact(case):
    torch, b = gpu()
    Xcal, X, W, bias, gr = layer_case(1, case["n"], case["P"], case["C"], 8, case["K"], case["bits"], case["dim"],
                                      case["om"], case["oc_"], case["ot"])
    g = b.calibrate_groups(to_dev(torch, Xcal), case["P"], case["bits"], case["K"], case["dim"], case["om"], 5.0)
    oracle_grouping_matches(gr, g.export())
    ref, _, _ = ol.quantize_static(X, gr, 0)
    Xq, _, _ = b.quantize_act(g, to_dev(torch, X))
    ex = g.export()
    got = unpermute_codes(Xq, ex["perm"], case["C"])
    assert np.array_equal(got, ref)
    # padding positions carry the zero-point of their cell (clamped to the code range)
    pads = np.flatnonzero(ex["perm"] < 0)
    if pads.size:
        Xq_h = Xq.cpu().numpy()
        grp = np.searchsorted(ex["group_off"], pads, side="right") - 1
        rows = np.arange(X.shape[0]) % case["P"]
        want = np.clip(gr.zp[0][gr.row_group[rows]][:, grp], 0, 2 ** case["bits"] - 1)
        assert np.array_equal(Xq_h[:, pads], want)
    assert b.device_status() == 0


@pytest.mark.parametrize("M,C,K,bits", [(256, 320, 4, 8), (1000, 1280, 8, 8), (77, 768, 16, 6), (3, 16, 2, 8)])
def test_dynamic_token_codes_bit_exact(M, C, K, bits):
    torch, b = gpu()
    Xcal, X, W, bias, gr = layer_case(2, 1, M, C, 8, K, bits, oc.DIM_CHANNEL)
    g = b.calibrate_groups(to_dev(torch, Xcal), M, bits, K, b.DIM_CHANNEL)
    ref, s_ref, z_ref = ol.quantize_dynamic_token(X, gr.col_group, gr.G, bits)
    Xq, ds, dz = b.quantize_act(g, to_dev(torch, X), mode=b.MODE_DYNAMIC_TOKEN)
    got = unpermute_codes(Xq, g.export()["perm"], C)
    assert np.array_equal(ds.cpu().numpy(), s_ref)
    assert np.array_equal(dz.cpu().numpy(), z_ref)
    assert np.array_equal(got, ref)
    assert b.device_status() == 0


def test_centred_layout_and_errors():
    torch, b = gpu()
    Xcal, X, W, bias, gr = layer_case(3, 2, 64, 64, 8, 4, 6, oc.DIM_CHANNEL, token_outliers=False)
    g = b.calibrate_groups(to_dev(torch, Xcal), 64, 6, 4, b.DIM_CHANNEL)
    ref, _, z = ol.quantize_static(X, gr, 0)
    Xq, _, _ = b.quantize_act(g, to_dev(torch, X), layout=b.CODES_S8_CENTRED)
    ex = g.export()
    got = unpermute_codes(Xq, ex["perm"], 64, signed=True)
    assert np.array_equal(got, ref - z[:, gr.col_group])
    assert np.all(Xq.cpu().numpy()[:, ex["perm"] < 0] == 0)
    Xd = to_dev(torch, X)
    with pytest.raises(b.DgqError) as e:
        b.quantize_act(g, Xd, timestep=5)
    assert e.value.status == 1
    with pytest.raises(b.DgqError) as e:       # misaligned base pointer
        b.quantize_act(g, Xd.view(-1)[4:4 + 64 * 4].view(4, 64))
    assert e.value.status == 2


def test_dynamic_token_degenerate_rows():
    """Rows whose groups are degenerate: all zeros, one constant (near and far from zero), the largest fp16
    magnitudes, a single spike.  A constant group takes the floor scale, so its zero-point leaves the code
    range (and, far from zero, the range where the kernel's conversion-free code path applies); codes, scales
    and zero-points must still match bit for bit, and the layer output must stay within tolerance through the
    epilogue's zero-point correction."""
    torch, b = gpu()
    M, C, N, K = 64, 320, 160, 4
    Xcal, X, W, bias, gr = layer_case(7, 1, M, C, N, K, 8, oc.DIM_CHANNEL)
    X = X.copy()
    X[0] = 0.0
    X[1] = 3.0
    X[2] = -5.0
    X[3] = 65504.0
    X[4] = -65504.0
    X[5] = 0.0
    X[5, 17] = 1000.0
    X[6, gr.col_group == 0] = 0.25                  # one constant group in an otherwise ordinary row
    X[7] = 6.1e-5                                   # the smallest normal fp16
    g = b.calibrate_groups(to_dev(torch, Xcal), M, 8, K, b.DIM_CHANNEL)
    ref, s_ref, z_ref = ol.quantize_dynamic_token(X, gr.col_group, gr.G, 8)
    Xq, ds, dz = b.quantize_act(g, to_dev(torch, X), mode=b.MODE_DYNAMIC_TOKEN)
    assert np.array_equal(ds.cpu().numpy(), s_ref)
    assert np.array_equal(dz.cpu().numpy(), z_ref)
    assert np.array_equal(unpermute_codes(Xq, g.export()["perm"], C), ref)
    wq, sw = ol.weight_rtn(W, 8)
    w = b.weight_prepare(g, to_dev(torch, W), 8)
    Y = b.linear(g, w, Xq, mode=b.MODE_DYNAMIC_TOKEN, dyn_scale=ds, dyn_zp=dz, bias=to_dev(torch, bias))
    assert b.device_status() == 0
    Yref = ol.group_linear(ref, s_ref, z_ref, gr.col_group, wq, sw, bias)
    Yg = Y.float().cpu().numpy().astype(np.float64)
    ordinary = np.ones(M, bool)
    ordinary[[3, 4]] = False                        # outputs beyond the fp16 range are compared apart
    assert np.max(np.abs(Yg[ordinary] - Yref[ordinary])) <= 1e-3 * np.max(np.abs(Yref[ordinary]))
    big = np.clip(Yref[~ordinary], -65504.0, 65504.0)
    got = np.nan_to_num(Yg[~ordinary], posinf=65504.0, neginf=-65504.0)
    assert np.max(np.abs(got - big)) <= 1e-3 * np.max(np.abs(big))


def test_nonfinite_inputs_static_both_code_paths():
    """NaN -> code 0, +inf -> the last code, -inf -> 0 (the fmax / fmin semantics of the fixed fp32 order), through
    the conversion-free code path (|Z| <= 2^21) and the canonical one (a zero-point far outside it), with tables
    handed over from the host.  Ordinary values around the specials must be unaffected."""
    torch, b = gpu()
    C, P, bits = 64, 16, 8
    col_group = (np.arange(C) // 16).astype(np.int32)                # 4 groups of 16 channels
    scale = np.array([[[0.05, 1e-6, 0.01, 2.0]]], np.float32)        # [T=1, R=1, G=4]
    zp = np.array([[[100, 5_000_000, -3_000_000, 255]]], np.int32)   # groups 1 and 2 are beyond 2^21
    g = b.groups_from_host(C, P, bits, col_group, np.zeros(P, np.int32), scale, zp)
    assert (g.G, g.R, g.T) == (4, 1, 1)
    rng = np.random.default_rng(5)
    X = rng.normal(0, 3, (48, C)).astype(np.float16)
    X[:, 16:32] = (5.0 + rng.normal(0, 1e-4, (48, 16))).astype(np.float16)      # near -Z s of group 1
    X[:, 32:48] = (-30000.0 + rng.normal(0, 50, (48, 16))).astype(np.float16)   # near -Z s of group 2
    for r, v in enumerate([np.nan, np.inf, -np.inf]):
        X[r::8, r::5] = v                                            # specials in every group and chunk position
    inv = (np.float32(1.0) / scale[0, 0]).astype(np.float32)
    ref = quantize_canonical_f32(X, inv[col_group][None, :], zp[0, 0][col_group][None, :], bits)
    assert set(np.unique(ref[np.isnan(X.astype(np.float32))])) == {0}
    assert set(np.unique(ref[np.isposinf(X.astype(np.float32))])) == {255}
    assert set(np.unique(ref[np.isneginf(X.astype(np.float32))])) == {0}
    Xq, _, _ = b.quantize_act(g, to_dev(torch, X))
    assert np.array_equal(unpermute_codes(Xq, g.export()["perm"], C), ref)
    assert b.device_status() == 0


def test_static_grid_at_8192_rows():
    """Both outlier types at the benchmark's size: 2 x 4096 tokens x 320 channels, a grid of pixel groups x
    channel groups; every code of the whole matrix against the oracle."""
    torch, b = gpu()
    P, C, K = 4096, 320, 4
    Xcal, X, W, bias, gr = layer_case(13, 2, P, C, 8, K, 8, oc.DIM_BOTH)
    g = b.calibrate_groups(to_dev(torch, Xcal), P, 8, K, b.DIM_BOTH)
    assert g.R > 1 and g.G > 1
    oracle_grouping_matches(gr, g.export())
    ref, _, _ = ol.quantize_static(X, gr, 0)
    Xq, _, _ = b.quantize_act(g, to_dev(torch, X))
    assert np.array_equal(unpermute_codes(Xq, g.export()["perm"], C), ref)
    assert b.device_status() == 0
