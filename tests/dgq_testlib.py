"""Helpers shared by the GPU parity tests: run the oracle and the CUDA library on the same seeded inputs."""
import os

import numpy as np
import pytest

from oracle import calibration as oc
from oracle import linear as ol
from paper_2501_04304_b200 import synth


def gpu():
    torch = pytest.importorskip("torch")
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2501_04304_b200 import binding
    return torch, binding


def to_dev(torch, a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def unpermute_codes(Xq, perm, C, signed=False):
    """Codes [M, K_pad] in the padded layout -> [M, C] in channel order."""
    Xq = Xq.cpu().numpy()
    if signed:
        Xq = Xq.view(np.int8)
    out = np.zeros((Xq.shape[0], C), dtype=np.int32)
    valid = perm >= 0
    out[:, perm[valid]] = Xq[:, valid]
    return out


def oracle_grouping_matches(gr, ex):
    """Same grouping and tables from the oracle (gr) and the library export (ex)."""
    assert np.array_equal(gr.col_group, ex["col_group"])
    assert np.array_equal(gr.row_group, ex["row_group"])
    for t in gr.scale:
        assert np.array_equal(gr.scale[t], ex["scale"][t])
        assert np.array_equal(gr.zp[t], ex["zp"][t])


def layer_case(seed, n_samples, P, C, N, K, bits, dim, outlier_mode=oc.OUTLIER_KMEANS,
               n_out_ch=None, n_out_tok=None, token_outliers=True, n_cal=4):
    Xcal = synth.activations(seed, 100, n_cal, P, C, n_out_ch, n_out_tok, token_outliers)
    X = synth.activations(seed, 1, n_samples, P, C, n_out_ch, n_out_tok, token_outliers)
    W = synth.weights(seed, 2, N, C)
    b = synth.bias(seed, 3, N)
    gr = oc.calibrate(Xcal, P, bits, K, dim_select=dim, outlier_mode=outlier_mode)
    return Xcal, X, W, b, gr


def check_output(Y_gpu, Y_ref, rel=1e-3):
    """fp16 layer output within rel * max|ref| of the fp64 oracle, element by element."""
    Yg = Y_gpu.float().cpu().numpy().astype(np.float64)
    err = np.max(np.abs(Yg - Y_ref))
    bound = rel * np.max(np.abs(Y_ref))
    assert err <= bound, f"max|delta| {err:.3e} > {rel} * max|ref| = {bound:.3e}"
    return err / np.max(np.abs(Y_ref))


CODE_FRAC = 1e-4   # log2 codes may differ from the oracle's by one level on at most this fraction of the entries


def check_codes(c, codes_ref):
    """Integer codes against the oracle's: never more than one level apart, and different on at most
    CODE_FRAC of the entries (rounded up to a whole entry, so the smallest cases tolerate one).  With
    DGQ_FLIP_REPORT set to a file name the measured counts are appended there.  Returns the absolute
    difference array."""
    diff = np.abs(np.asarray(c, dtype=np.int64) - np.asarray(codes_ref, dtype=np.int64))
    assert diff.max() <= 1, "a code differs by more than one level"
    n_flips = int((diff != 0).sum())
    path = os.environ.get("DGQ_FLIP_REPORT")
    if path:
        with open(path, "a") as fh:
            fh.write(f"{os.environ.get('PYTEST_CURRENT_TEST', '')} entries {diff.size} flips {n_flips}\n")
    allowed = int(np.ceil(CODE_FRAC * diff.size))
    assert n_flips <= allowed, f"{n_flips} of {diff.size} codes differ (allowed {allowed})"
    return diff


def flipped_output_bound(diff, c, codes_ref, s, V_rest):
    """How far a row's output may move when some of its codes sit one level off: an entry whose code is c
    instead of c +- 1 changes its weight s 2^-code by s 2^-max(codes), times |V_j| per feature.
    diff, c, codes_ref [B, H, nq, n]; s broadcastable to them; V_rest [B, n, H, d] -> bound [B, nq, H, d]."""
    w = np.where(diff != 0, np.ldexp(np.broadcast_to(s, diff.shape).astype(np.float64),
                                     -np.maximum(c, codes_ref).astype(np.int64)), 0.0)
    return np.einsum("bhqk,bkhd->bqhd", w, np.abs(np.asarray(V_rest, dtype=np.float64)))
