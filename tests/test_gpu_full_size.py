"""GPU parity at the sizes and launch configurations the benchmark times (persistent kernels, several tiles
per CTA, every SM busy): outputs are checked on sampled rows that the oracle computes one by one."""
import numpy as np
import pytest

from oracle import calibration as oc
from oracle import linear as ol
from paper_2501_04304_b200 import synth
from dgq_testlib import gpu, to_dev, unpermute_codes, check_codes, flipped_output_bound
from test_gpu_attention import _compare
from oracle import attention as oa

pytestmark = pytest.mark.gpu

REL = 1e-3


def _sample_rows(M, seed):
    rng = np.random.default_rng(seed)
    fixed = [0, 1, 127, 128, 129, 255, 256, M // 2 - 1, M // 2, M - 129, M - 128, M - 2, M - 1]
    rows = np.unique(np.concatenate([np.asarray(fixed), rng.integers(0, M, 64)]))
    return rows[(rows >= 0) & (rows < M)]


@pytest.mark.parametrize("P,batch,C,N,w_bits", [
    (4096, 2, 320, 2560, 8),     # FF1 of the 64 x 64 level: 64 x 16 tiles on 144 CTAs
    (4096, 2, 1280, 320, 8),     # FF2: long K, two column blocks
    (4096, 2, 320, 960, 8),      # stacked q/k/v projection
    (1024, 8, 640, 640, 4),      # 32 x 32 level, 4-bit weights
    # 4-bit weights over every transformer linear of the four UNet levels at batch 8: q/k/v/out (ch -> ch),
    # the gated feed-forward (ch -> 8 ch, 4 ch -> ch) and the cross-attention k/v projections of the 77
    # context tokens (768 -> ch)
    (4096, 8, 320, 320, 4), (4096, 8, 320, 2560, 4), (4096, 8, 1280, 320, 4), (77, 8, 768, 320, 4),
    (1024, 8, 640, 5120, 4), (1024, 8, 2560, 640, 4), (77, 8, 768, 640, 4),
    (256, 8, 1280, 1280, 4), (256, 8, 1280, 10240, 4), (256, 8, 5120, 1280, 4), (77, 8, 768, 1280, 4),
    (64, 8, 1280, 1280, 4), (64, 8, 1280, 10240, 4), (64, 8, 5120, 1280, 4),
    # the second model of Table 2 (SDXL-Turbo at 512 x 512, one image): transformer levels of 1024 tokens x
    # 640 channels and 256 tokens x 1280 channels, context of 77 tokens x 2048
    (1024, 1, 640, 640, 8), (1024, 1, 640, 5120, 8), (1024, 1, 2560, 640, 8), (77, 1, 2048, 640, 8),
    (256, 1, 1280, 1280, 8), (256, 1, 1280, 10240, 4), (256, 1, 5120, 1280, 4), (77, 1, 2048, 1280, 4),
])
def test_linear_full_size_sampled_rows(P, batch, C, N, w_bits):
    torch, b = gpu()
    M = P * batch
    Xcal = synth.activations(21, 100, 4, P, C)
    X = synth.activations(21, 1, batch, P, C)
    W = synth.weights(21, 2, N, C)
    bias = synth.bias(21, 3, N)
    gr = oc.calibrate(Xcal, P, 8, 8, dim_select=oc.DIM_CHANNEL)
    g = b.calibrate_groups(to_dev(torch, Xcal), P, 8, 8, b.DIM_CHANNEL)
    wq, sw = ol.weight_rtn(W, w_bits)
    w = b.weight_prepare(g, to_dev(torch, W), w_bits)
    Xq, ds, dz = b.quantize_act(g, to_dev(torch, X), mode=b.MODE_DYNAMIC_TOKEN)
    Y = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")   # a tile left unwritten stays NaN
    b.linear(g, w, Xq, mode=b.MODE_DYNAMIC_TOKEN, dyn_scale=ds, dyn_zp=dz, bias=to_dev(torch, bias), out=Y)
    torch.cuda.synchronize()
    assert b.device_status() == 0
    rows = _sample_rows(M, 5)
    codes, s_rows, z_rows = ol.quantize_dynamic_token(X[rows], gr.col_group, gr.G, gr.bits)
    got_codes = unpermute_codes(Xq[torch.from_numpy(rows).cuda()], g.export()["perm"], C)
    assert np.array_equal(got_codes, codes)                      # integer work: bit-exact
    Yref = ol.group_linear(codes, s_rows, z_rows, gr.col_group, wq, sw, bias)
    Yg = Y[torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
    err = np.max(np.abs(Yg - Yref))
    assert err <= REL * np.max(np.abs(Yref)), f"max|delta| {err:.3e} on sampled rows"
    assert np.isfinite(Y.float().cpu().numpy()).all()            # every tile was written


@pytest.mark.parametrize("C,N", [(320, 320), (320, 960), (320, 2560), (1280, 320)])
def test_config2_whole_output(C, N):
    """The W8A8 linears of the 64 x 64 transformer level at batch 2 (8192 tokens; q/k/v stacked to 960 outputs):
    every output element against the oracle, per-token dynamic scales, output pre-filled with NaN."""
    torch, b = gpu()
    P, batch = 4096, 2
    M = P * batch
    Xcal = synth.activations(25, 100, 4, P, C)
    X = synth.activations(25, 1, batch, P, C)
    W = synth.weights(25, 2, N, C)
    bias = synth.bias(25, 3, N)
    gr = oc.calibrate(Xcal, P, 8, 8, dim_select=oc.DIM_CHANNEL)
    g = b.calibrate_groups(to_dev(torch, Xcal), P, 8, 8, b.DIM_CHANNEL)
    wq, sw = ol.weight_rtn(W, 8)
    w = b.weight_prepare(g, to_dev(torch, W), 8)
    Xq, ds, dz = b.quantize_act(g, to_dev(torch, X), mode=b.MODE_DYNAMIC_TOKEN)
    Y = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    b.linear(g, w, Xq, mode=b.MODE_DYNAMIC_TOKEN, dyn_scale=ds, dyn_zp=dz, bias=to_dev(torch, bias), out=Y)
    torch.cuda.synchronize()
    assert b.device_status() == 0
    codes, s_rows, z_rows = ol.quantize_dynamic_token(X, gr.col_group, gr.G, gr.bits)
    assert np.array_equal(unpermute_codes(Xq, g.export()["perm"], C), codes)
    Yref = ol.group_linear(codes, s_rows, z_rows, gr.col_group, wq, sw, bias)
    Yg = Y.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(Yg).all()
    err = np.max(np.abs(Yg - Yref))
    assert err <= REL * np.max(np.abs(Yref)), f"max|delta| {err:.3e}"


def test_static_mode_full_size_linear():
    """Static tables (the paper's mode) at 8192 x 320 -> 2560 with both pixel and channel groups: sampled rows
    against the oracle, every tile written."""
    torch, b = gpu()
    P, batch, C, N = 4096, 2, 320, 2560
    M = P * batch
    Xcal = synth.activations(26, 100, 4, P, C)
    X = synth.activations(26, 1, batch, P, C)
    W = synth.weights(26, 2, N, C)
    bias = synth.bias(26, 3, N)
    gr = oc.calibrate(Xcal, P, 8, 4, dim_select=oc.DIM_BOTH)
    g = b.calibrate_groups(to_dev(torch, Xcal), P, 8, 4, b.DIM_BOTH)
    assert g.R > 1 and g.G > 1
    wq, sw = ol.weight_rtn(W, 8)
    w = b.weight_prepare(g, to_dev(torch, W), 8)
    Xq, _, _ = b.quantize_act(g, to_dev(torch, X))
    Y = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    b.linear(g, w, Xq, bias=to_dev(torch, bias), out=Y)
    torch.cuda.synchronize()
    assert b.device_status() == 0
    rows = _sample_rows(M, 6)
    rows = np.unique(np.concatenate([rows, np.flatnonzero(gr.row_group > 0)[:8]]))   # rows of the outlier pixel groups too
    codes, s_all, z_all = ol.quantize_static(X, gr, 0)
    Yref = ol.group_linear(codes[rows], s_all[rows], z_all[rows], gr.col_group, wq, sw, bias)
    Yg = Y[torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
    assert np.max(np.abs(Yg - Yref)) <= REL * np.max(np.abs(Yref))
    assert np.isfinite(Y.float().cpu().numpy()).all()


@pytest.mark.parametrize("n,H,Wd,C", [
    (2, 64, 64, 320),            # the benchmark's launch
    (8, 64, 64, 320), (8, 32, 32, 640), (8, 16, 16, 1280), (8, 8, 8, 1280),   # the four levels at batch 8
])
def test_conv_full_size_sampled_bands(n, H, Wd, C):
    """3 x 3 conv C -> C, W4A6, 16 groups: image-border and interior bands of output rows of the first, second
    and last image."""
    torch, b = gpu()
    N, K = C, 16
    P = H * Wd
    Xcal = synth.activations(22, 100, 4, P, C, None, None, token_outliers=False)
    X = synth.activations(22, 1, n, P, C, None, None, token_outliers=False)
    Wt = synth.conv_weights(22, 2, N, C)
    bias = synth.bias(22, 3, N)
    gr = oc.calibrate(Xcal, P, 6, K, dim_select=oc.DIM_CHANNEL)
    g = b.calibrate_groups(to_dev(torch, Xcal), P, 6, K, b.DIM_CHANNEL)
    wq, sw = ol.weight_rtn(Wt, 4)
    conv = (n, H, Wd, C)
    w = b.weight_prepare(g, to_dev(torch, Wt), 4, conv=conv)
    Xq, _, _ = b.quantize_act(g, to_dev(torch, X), layout=b.CODES_S8_CENTRED)
    Y = torch.full((n * P, N), float("nan"), dtype=torch.float16, device="cuda")  # a tile left unwritten stays NaN
    b.linear(g, w, Xq, layout=b.CODES_S8_CENTRED, bias=to_dev(torch, bias), conv=conv, out=Y)
    torch.cuda.synchronize()
    assert b.device_status() == 0
    Yg = Y.float().cpu().numpy().astype(np.float64).reshape(n, H, Wd, N)
    codes, _, _ = ol.quantize_static(X, gr, 0)
    codes = codes.reshape(n, H, Wd, C)
    worst, ref_max = 0.0, 0.0
    mid = H // 2
    for img, h0, h1 in [(0, 0, 2), (0, mid - 1, mid + 1), (0, H - 2, H), (1, 0, 1), (1, 1, 3), (1, H - 1, H),
                        (n - 1, 0, 1), (n - 1, mid, mid + 1), (n - 1, H - 1, H)]:
        lo, hi = max(h0 - 1, 0), min(h1 + 1, H)                  # the band with the rows it reads
        sub = ol.group_conv3x3(codes[img:img + 1, lo:hi], gr.scale[0][0], gr.zp[0][0], gr.col_group, wq, sw, bias)
        ref = sub[0, h0 - lo:h0 - lo + (h1 - h0)]                # rows whose neighbours are real rows or the border
        worst = max(worst, np.max(np.abs(Yg[img, h0:h1] - ref)))
        ref_max = max(ref_max, np.max(np.abs(ref)))
    assert worst <= REL * ref_max, f"max|delta| {worst:.3e} vs max|ref| {ref_max:.3e}"
    assert np.isfinite(Yg).all()


@pytest.mark.parametrize("nq,d,bits", [(4096, 40, 8), (4096, 40, 4), (1024, 80, 8), (256, 160, 8), (64, 160, 8),
                                       (64, 160, 4)])
def test_attention_full_size(nq, d, bits):
    """B 2, H 8, nk 77 at the four UNet levels (nq x d = 4096 x 40 ... 64 x 160): the whole output against
    the oracle."""
    torch, b = gpu()
    Q, K, V = synth.attention_inputs(23, 2, 8, nq, 77, d)
    _compare(torch, b, Q, K, V, bits)


@pytest.mark.parametrize("H,nq", [(10, 1024), (20, 256)])
def test_attention_sdxl_turbo_levels(H, nq):
    """Heads of 64 features (640 / 10 and 1280 / 20 channels), context projected from 2048 features."""
    torch, b = gpu()
    Q, K, V = synth.attention_inputs(24, 1, H, nq, 77, 64, ctx_dim=2048)
    _compare(torch, b, Q, K, V, 8)


def test_self_attention_full_size_sampled_rows():
    """4096 tokens attending to 4096 keys (the 64 x 64 level): every query row is independent with a per-row
    scale, so the oracle computes sampled rows against all keys and those rows are compared in full."""
    torch, b = gpu()
    B, H, n, d = 2, 8, 4096, 40
    rng = np.random.default_rng(41)
    Q = rng.normal(0, 1, (B, n, H, d)).astype(np.float16)
    K = rng.normal(0, 1, (B, n, H, d)).astype(np.float16)
    V = rng.normal(0, 1, (B, n, H, d)).astype(np.float16)
    O, codes = b.self_attn_logq(to_dev(torch, Q), to_dev(torch, K), to_dev(torch, V), 8, want_codes=True)
    torch.cuda.synchronize()
    assert b.device_status() == 0
    rows = _sample_rows(n, 5)[::2]
    O_ref, codes_ref, s_ref, _ = oa.self_attn_logq(Q[:, rows], K, V, 8)
    c = codes[:, :, torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.int64)
    diff = check_codes(c, codes_ref)
    O_alt = oa.self_product(c, s_ref, V)
    Og = O[:, torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
    assert np.max(np.abs(Og - O_alt)) <= REL * np.max(np.abs(O_alt))
    bound = REL * np.max(np.abs(O_ref)) + flipped_output_bound(diff, c, codes_ref, s_ref, V)
    assert np.all(np.abs(Og - O_ref) <= bound)


def test_chained_layers_in_a_graph_match_serialised_calls():
    """Back-to-back dependent kernels (quantize -> linear -> quantize -> linear -> attention on the result)
    replayed as one CUDA graph give bit for bit what the same calls give with a device synchronisation after
    each: the kernels are launched so that a kernel may be scheduled while its predecessor drains, and each
    must wait for its predecessor's writes before it reads or writes anything."""
    torch, b = gpu()
    P, batch, C = 4096, 2, 320
    M = P * batch
    Xcal = synth.activations(31, 100, 4, P, C)
    X = to_dev(torch, synth.activations(31, 1, batch, P, C))
    g = b.calibrate_groups(to_dev(torch, Xcal), P, 8, 8, b.DIM_CHANNEL)
    w1 = b.weight_prepare(g, to_dev(torch, synth.weights(31, 2, C, C)), 8)
    w2 = b.weight_prepare(g, to_dev(torch, synth.weights(31, 3, C, C)), 8)
    B, H, nq, nk, d = 2, 8, 4096, 77, 40
    _, Kc, Vc = synth.attention_inputs(31, B, H, nq, nk, d)
    Kd, Vd = to_dev(torch, Kc), to_dev(torch, Vc)

    def buffers():
        return dict(xq=torch.empty((M, g.K_pad), dtype=torch.uint8, device="cuda"),
                    ds=torch.empty((M, g.G), dtype=torch.float32, device="cuda"),
                    dz=torch.empty((M, g.G), dtype=torch.int32, device="cuda"),
                    y1=torch.empty((M, C), dtype=torch.float16, device="cuda"),
                    y2=torch.empty((M, C), dtype=torch.float16, device="cuda"),
                    o=torch.empty((B, nq, H, d), dtype=torch.float16, device="cuda"),
                    ws=torch.empty(b.cross_attn_workspace_bytes(B, H, nq, nk, d), dtype=torch.uint8, device="cuda"))

    def chain(t, sync):
        def s():
            if sync:
                torch.cuda.synchronize()
        b.quantize_act_into(g, X, t["xq"], t["ds"], t["dz"], mode=b.MODE_DYNAMIC_TOKEN); s()
        b.linear(g, w1, t["xq"], mode=b.MODE_DYNAMIC_TOKEN, dyn_scale=t["ds"], dyn_zp=t["dz"], out=t["y1"]); s()
        b.quantize_act_into(g, t["y1"], t["xq"], t["ds"], t["dz"], mode=b.MODE_DYNAMIC_TOKEN); s()   # reuses the buffers
        b.linear(g, w2, t["xq"], mode=b.MODE_DYNAMIC_TOKEN, dyn_scale=t["ds"], dyn_zp=t["dz"], out=t["y2"]); s()
        q = t["y2"].view(B, nq, H, d)                                                                  # 8192 x 320
        b.cross_attn_logq(q, Kd, Vd, 8, out=t["o"], workspace=t["ws"]); s()

    ref = buffers()
    chain(ref, sync=True)
    torch.cuda.synchronize()
    got = buffers()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        chain(got, sync=False)                       # warm-up outside the capture
        stream.synchronize()
        for v in got.values():
            v.zero_()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            chain(got, sync=False)
        for _ in range(3):
            graph.replay()
    torch.cuda.synchronize()
    assert b.device_status() == 0
    for k in ("y1", "y2", "o"):
        assert torch.equal(got[k], ref[k]), k
