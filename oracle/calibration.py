"""Outlier-preserving group calibration, Sec. 3.3 (Eq. 4 - Eq. 7).

Test infrastructure only; see the package docstring.

An activation matrix of one layer at one timestep is viewed as
[n_samples * P, C]: P pixels (tokens) per sample, C channels.  "The i-th
vector in dimension d" (Eq. 4) is read as: d = channel -> column i over all
rows; d = pixel -> pixel position i (row index mod P) over all channels and
samples, since the paper reports that outlier pixels stay at the same positions
across prompts and seeds (Sec. 3.2).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from .quantizers import group_params_array

DIM_AUTO, DIM_CHANNEL, DIM_PIXEL, DIM_BOTH = 0, 1, 2, 3
OUTLIER_KMEANS, OUTLIER_EXPLICIT = 0, 1


def vector_extrema(X, P):
    """Per-channel and per-pixel (min, max) of X [n*P, C] (Eq. 4's a^min, a^max)."""
    X = np.asarray(X, dtype=np.float64)
    n = X.shape[0] // P
    assert n * P == X.shape[0]
    ch_min, ch_max = X.min(axis=0), X.max(axis=0)
    Xp = X.reshape(n, P, X.shape[1])
    px_min, px_max = Xp.min(axis=(0, 2)), Xp.max(axis=(0, 2))
    return ch_min, ch_max, px_min, px_max


def range_variability(vmin, vmax):
    """Eq. 4: spread of the per-vector maxima plus spread of the per-vector minima."""
    return (np.max(vmax) - np.min(vmax)) + (np.max(vmin) - np.min(vmin))


def select_dimension(D_channel, D_pixel):
    """Eq. 5: the dimension with the larger D_d; a tie goes to channel (first argument)."""
    return DIM_CHANNEL if D_channel >= D_pixel else DIM_PIXEL


def kmeans_ranges(vmin, vmax, K, max_iter=100):
    """K groups of vectors "based on their range" (Sec. 3.3, before Eq. 6).

    The paper names K-means and nothing else.  Reading: each vector is the 2-D
    point (min_i, max_i); plain Lloyd iterations with squared Euclidean
    distance, made deterministic as follows (parity unpinned: any such choice
    is defensible): vectors are ranked by width max - min (stable, index breaks
    ties) and centroid k starts at the vector of rank floor((2k+1) n / (2K));
    a point goes to its nearest centroid (lowest k on ties); means are summed in
    index order in fp64; iteration stops when the assignment repeats or after
    `max_iter` rounds; a cluster that loses all members keeps its centroid and
    is dropped at the end; the surviving groups are renumbered by ascending
    centroid width.  Returns int labels in [0, G_eff).
    """
    vmin = np.asarray(vmin, dtype=np.float64)
    vmax = np.asarray(vmax, dtype=np.float64)
    n = vmin.shape[0]
    K = max(1, min(int(K), n))
    width = vmax - vmin
    order = sorted(range(n), key=lambda i: (width[i], i))
    cx = np.empty(K)
    cy = np.empty(K)
    for k in range(K):
        i = order[((2 * k + 1) * n) // (2 * K)]
        cx[k], cy[k] = vmin[i], vmax[i]
    labels = None
    for _ in range(max_iter):
        dx = vmin[:, None] - cx[None, :]
        dy = vmax[:, None] - cy[None, :]
        new = np.argmin(dx * dx + dy * dy, axis=1)      # first minimum -> lowest k
        if labels is not None and np.array_equal(new, labels):
            break
        labels = new
        sx = [0.0] * K
        sy = [0.0] * K
        cnt = [0] * K
        for i in range(n):                               # index order within every cluster
            k = int(labels[i])
            sx[k] += float(vmin[i])
            sy[k] += float(vmax[i])
            cnt[k] += 1
        for k in range(K):
            if cnt[k]:
                cx[k], cy[k] = sx[k] / cnt[k], sy[k] / cnt[k]
    used = [k for k in range(K) if np.any(labels == k)]
    used.sort(key=lambda k: (cy[k] - cx[k], k))
    remap = {k: j for j, k in enumerate(used)}
    return np.array([remap[int(k)] for k in labels], dtype=np.int32)


def explicit_outliers(vmin, vmax, tau):
    """Vectors whose range width exceeds tau x the median width.

    Not in the paper: a reading of the benchmark configuration that asks for
    "channel groups plus an outlier group".  The median of an even count is the
    mean of the two middle widths.
    """
    width = np.asarray(vmax, dtype=np.float64) - np.asarray(vmin, dtype=np.float64)
    return width > float(tau) * float(np.median(width))


def group_vectors(vmin, vmax, K, outlier_mode=OUTLIER_KMEANS, tau=5.0):
    """Group labels along one dimension.

    OUTLIER_KMEANS: K-means with K groups on all vectors (the paper).
    OUTLIER_EXPLICIT: the explicit outliers form one extra, last group and
    K-means with K groups runs on the rest.
    """
    vmin = np.asarray(vmin, dtype=np.float64)
    vmax = np.asarray(vmax, dtype=np.float64)
    if outlier_mode == OUTLIER_KMEANS:
        return kmeans_ranges(vmin, vmax, K)
    out = explicit_outliers(vmin, vmax, tau)
    labels = np.empty(vmin.shape[0], dtype=np.int32)
    rest = np.flatnonzero(~out)
    g_rest = 0
    if rest.size:
        lr = kmeans_ranges(vmin[rest], vmax[rest], K)
        labels[rest] = lr
        g_rest = int(lr.max()) + 1
    labels[np.flatnonzero(out)] = g_rest
    return labels


@dataclass
class Grouping:
    """Grouping of one layer (fixed) and its per-timestep (s, inv_s, Z) tables (Eq. 7)."""
    C: int
    P: int
    bits: int
    dim: int                      # DIM_CHANNEL, DIM_PIXEL or DIM_BOTH actually used
    col_group: np.ndarray         # [C] -> g
    row_group: np.ndarray         # [P] -> r
    G: int
    R: int
    D_channel: float = 0.0
    D_pixel: float = 0.0
    scale: dict = field(default_factory=dict)      # t -> float32 [R, G]
    inv_scale: dict = field(default_factory=dict)  # t -> float32 [R, G]
    zp: dict = field(default_factory=dict)         # t -> int32   [R, G]


def cell_extrema(X, P, row_group, R, col_group, G):
    """(lo, hi) of every (row group, column group) cell of X [n*P, C]; empty cells get (0, 0)."""
    X = np.asarray(X, dtype=np.float64)
    n = X.shape[0] // P
    rg = np.tile(np.asarray(row_group), n)
    lo = np.zeros((R, G))
    hi = np.zeros((R, G))
    for r in range(R):
        rows = X[rg == r]
        for g in range(G):
            cell = rows[:, np.asarray(col_group) == g]
            if cell.size:
                lo[r, g], hi[r, g] = cell.min(), cell.max()
    return lo, hi


def fill_timestep(gr: Grouping, X, timestep):
    """Eq. 6 for every cell from this timestep's calibration rows; one row of Eq. 7's sets."""
    lo, hi = cell_extrema(X, gr.P, gr.row_group, gr.R, gr.col_group, gr.G)
    s, inv_s, Z = group_params_array(lo, hi, gr.bits)
    gr.scale[timestep], gr.inv_scale[timestep], gr.zp[timestep] = s, inv_s, Z
    return gr


def calibrate(X, P, bits, K, dim_select=DIM_AUTO, outlier_mode=OUTLIER_KMEANS,
              tau=5.0, timestep=0) -> Grouping:
    """First calibration call of a layer: choose d* (Eq. 4, 5), group, fill one table row.

    The grouping is fixed per layer from then on and only (s, Z) change with the
    timestep: the paper's parameter-memory figure counts T x groups scalars and
    no per-timestep index maps (Sec. 3.3, after Eq. 7).  DIM_BOTH groups along
    both dimensions independently and gives every (pixel group, channel group)
    cell its own range - a group per outlier type (Sec. 1).
    """
    X = np.asarray(X)
    C = X.shape[1]
    ch_min, ch_max, px_min, px_max = vector_extrema(X, P)
    Dc = range_variability(ch_min, ch_max)
    Dp = range_variability(px_min, px_max)
    dim = select_dimension(Dc, Dp) if dim_select == DIM_AUTO else dim_select
    col_group = np.zeros(C, dtype=np.int32)
    row_group = np.zeros(P, dtype=np.int32)
    if dim in (DIM_CHANNEL, DIM_BOTH):
        col_group = group_vectors(ch_min, ch_max, K, outlier_mode, tau)
    if dim in (DIM_PIXEL, DIM_BOTH):
        row_group = group_vectors(px_min, px_max, K, outlier_mode, tau)
    gr = Grouping(C=C, P=P, bits=bits, dim=dim, col_group=col_group, row_group=row_group,
                  G=int(col_group.max()) + 1, R=int(row_group.max()) + 1,
                  D_channel=float(Dc), D_pixel=float(Dp))
    return fill_timestep(gr, X, timestep)
