"""Pins for the oracle's calibration (Eq. 4 - Eq. 7): closed forms, special cases, a library K-means."""
import numpy as np
import pytest

from oracle import calibration as oc
from oracle import quantizers as oq
from paper_2501_04304_b200 import synth


def test_Dd_hand_3x3():
    # rows = pixels, columns = channels
    X = np.array([[1.0, -2.0, 3.0],
                  [0.5, 9.0, -1.0],
                  [-4.0, 0.0, 2.0]])
    ch_min, ch_max, px_min, px_max = oc.vector_extrema(X, 3)
    assert ch_max.tolist() == [1.0, 9.0, 3.0] and ch_min.tolist() == [-4.0, -2.0, -1.0]
    assert px_max.tolist() == [3.0, 9.0, 2.0] and px_min.tolist() == [-2.0, -1.0, -4.0]
    # D_channel = (9 - 1) + (-1 - -4) = 11 ; D_pixel = (9 - 2) + (-1 - -4) = 10
    assert oc.range_variability(ch_min, ch_max) == 11.0
    assert oc.range_variability(px_min, px_max) == 10.0
    assert oc.select_dimension(11.0, 10.0) == oc.DIM_CHANNEL
    assert oc.select_dimension(10.0, 10.0) == oc.DIM_CHANNEL      # tie -> first
    assert oc.select_dimension(1.0, 10.0) == oc.DIM_PIXEL


def test_pixel_extrema_pool_samples():
    # two samples of P = 2 pixels: pixel position p pools rows p and p + P
    X = np.array([[1.0, 2.0], [3.0, 4.0], [-5.0, 0.0], [7.0, 1.0]])
    _, _, px_min, px_max = oc.vector_extrema(X, 2)
    assert px_min.tolist() == [-5.0, 1.0] and px_max.tolist() == [2.0, 7.0]


def test_dimension_follows_outlier_type():
    rng = np.random.default_rng(0)
    base = rng.standard_normal((4 * 64, 48))
    Xc = base.copy(); Xc[:, [3, 17]] *= 30
    Xp = base.copy(); Xp[np.arange(4 * 64) % 64 == 5] *= 30
    assert oc.calibrate(Xc, 64, 8, 4).dim == oc.DIM_CHANNEL
    assert oc.calibrate(Xp, 64, 8, 4).dim == oc.DIM_PIXEL


def _sse(vmin, vmax, labels):
    t = 0.0
    for k in np.unique(labels):
        m = labels == k
        t += ((vmin[m] - vmin[m].mean()) ** 2 + (vmax[m] - vmax[m].mean()) ** 2).sum()
    return t


def test_kmeans_special_cases():
    rng = np.random.default_rng(1)
    vmax = np.abs(rng.standard_normal(100)) + 1
    vmin = -np.abs(rng.standard_normal(100)) - 1
    assert np.all(oc.kmeans_ranges(vmin, vmax, 1) == 0)                    # K = 1: one group
    # K >= number of distinct points: every distinct point its own cluster, zero SSE
    pts_min = np.array([-1.0, -1.0, -2.0, -5.0, -2.0])
    pts_max = np.array([1.0, 1.0, 2.0, 5.0, 2.0])
    lab = oc.kmeans_ranges(pts_min, pts_max, 5)
    assert _sse(pts_min, pts_max, lab) == 0.0
    assert lab[0] == lab[1] and lab[2] == lab[4] and len(set(lab.tolist())) == 3
    # groups are numbered by ascending width
    assert lab[0] < lab[2] < lab[3]


def test_kmeans_recovers_separated_clusters():
    rng = np.random.default_rng(2)
    centres = [(-1, 1), (-4, 4), (-30, 30), (-1, 25)]
    truth = rng.integers(0, 4, 300)
    vmin = np.array([centres[t][0] for t in truth]) + rng.uniform(-0.2, 0.2, 300)
    vmax = np.array([centres[t][1] for t in truth]) + rng.uniform(-0.2, 0.2, 300)
    lab = oc.kmeans_ranges(vmin, vmax, 4)
    # same partition
    for t in range(4):
        assert len(set(lab[truth == t].tolist())) == 1
    assert len(set(lab.tolist())) == 4


def test_kmeans_matches_library_lloyd():
    """Same initial centroids -> scikit-learn's Lloyd iterations reach the same partition."""
    sklearn = pytest.importorskip("sklearn.cluster")
    rng = np.random.default_rng(3)
    n, K = 400, 6
    width = np.concatenate([rng.uniform(2, 3, 250), rng.uniform(6, 8, 100), rng.uniform(40, 60, 50)])
    mid = rng.normal(0, 0.3, n)
    vmin, vmax = mid - width / 2, mid + width / 2
    lab = oc.kmeans_ranges(vmin, vmax, K)
    order = sorted(range(n), key=lambda i: (vmax[i] - vmin[i], i))
    init = np.array([[vmin[order[((2 * k + 1) * n) // (2 * K)]],
                      vmax[order[((2 * k + 1) * n) // (2 * K)]]] for k in range(K)])
    km = sklearn.KMeans(n_clusters=K, init=init, n_init=1, algorithm="lloyd", max_iter=100, tol=0.0)
    ref = km.fit_predict(np.stack([vmin, vmax], axis=1))
    pairs = set(zip(lab.tolist(), ref.tolist()))
    assert len(pairs) == len(set(lab.tolist())) == len(set(ref.tolist()))      # a bijection of labels
    # Lloyd never increases the SSE
    init_lab = np.argmin(((np.stack([vmin, vmax], 1)[:, None, :] - init[None]) ** 2).sum(-1), axis=1)
    assert _sse(vmin, vmax, lab) <= _sse(vmin, vmax, init_lab) + 1e-9


def test_calibration_invariants_config1():
    X = synth.activations(0, 100, 4, 256, 320, n_out_ch=4, n_out_tok=2)
    gr = oc.calibrate(X, 256, 8, 4, dim_select=oc.DIM_BOTH, outlier_mode=oc.OUTLIER_EXPLICIT)
    out_c = synth.outlier_channels(0, 320, 4)
    out_t = synth.outlier_tokens(0, 256, 2)
    assert gr.G == 5 and gr.R >= 2
    # the outlier channels form the last group, alone
    assert set(np.flatnonzero(gr.col_group == gr.G - 1).tolist()) == set(out_c.tolist())
    assert set(np.flatnonzero(gr.row_group == gr.R - 1).tolist()) == set(out_t.tolist())
    # every vector in exactly one group; every cell's range contains its members
    assert gr.col_group.min() == 0 and gr.col_group.max() == gr.G - 1
    Xf = X.astype(np.float64)
    rg = np.tile(gr.row_group, 4)
    s, Z = gr.scale[0], gr.zp[0]
    for r in range(gr.R):
        for g in range(gr.G):
            cell = Xf[rg == r][:, gr.col_group == g]
            lo_rep = float(s[r, g]) * (0 - int(Z[r, g]))
            hi_rep = float(s[r, g]) * (2 ** 8 - int(Z[r, g]))
            assert cell.min() >= lo_rep - float(s[r, g]) and cell.max() <= hi_rep + float(s[r, g])
            assert float(s[r, g]) == float(np.float32((np.float32(cell.max()) - np.float32(cell.min()))) * np.float32(2.0 ** -8))


def test_one_group_is_layerwise_minmax():
    """G = 1, R = 1 equals layer-wise asymmetric MinMax quantization, written independently."""
    from oracle import linear as ol
    X = synth.activations(3, 7, 2, 32, 24, n_out_ch=1, n_out_tok=1)
    gr = oc.calibrate(X, 32, 8, 1, dim_select=oc.DIM_CHANNEL)
    assert gr.G == 1 and gr.R == 1
    codes, _, _ = ol.quantize_static(X, gr, 0)
    xs = [float(v) for v in X.astype(np.float32).ravel()]
    lo, hi = np.float32(min(xs)), np.float32(max(xs))
    s = np.float32(np.float32(hi - lo) / np.float32(256.0))
    inv = np.float32(1.0) / s
    z = int(np.rint(np.float32(-lo * inv)))
    ref = [int(min(max(np.rint(np.float32(np.float32(v) * inv)) + z, 0), 255)) for v in xs]
    assert codes.ravel().tolist() == ref


def test_group_per_channel_is_channelwise():
    from oracle import linear as ol
    X = synth.activations(4, 8, 2, 16, 12, n_out_ch=2, n_out_tok=1)
    gr = oc.calibrate(X, 16, 6, 12, dim_select=oc.DIM_CHANNEL)
    Xf = X.astype(np.float32)
    if gr.G == 12:                                   # every channel its own group
        codes, _, _ = ol.quantize_static(X, gr, 0)
        for c in range(12):
            s, inv, z = oq.group_params(Xf[:, c].min(), Xf[:, c].max(), 6)
            assert np.array_equal(codes[:, c], oq.quantize_canonical_f32(Xf[:, c], inv, z, 6))
    else:                                            # duplicates merged: still one range per distinct point
        assert gr.G < 12


def test_timestep_rows_share_grouping():
    X0 = synth.activations(5, 1, 2, 32, 24, n_out_ch=1, n_out_tok=1)
    X1 = (synth.activations(5, 2, 2, 32, 24, n_out_ch=1, n_out_tok=1).astype(np.float32) * 2).astype(np.float16)
    gr = oc.calibrate(X0, 32, 8, 3, dim_select=oc.DIM_CHANNEL, timestep=0)
    cg = gr.col_group.copy()
    oc.fill_timestep(gr, X1, 1)
    assert np.array_equal(cg, gr.col_group)
    assert set(gr.scale) == {0, 1}
    assert np.all(gr.scale[1] > gr.scale[0])
