"""Thin ctypes binding of the C-ABI library declared in include/dgq.h.

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  Tensors are torch CUDA tensors (device memory and streams come from
PyTorch); their data pointers go to the library as plain pointers.  Loading
fails loudly when the library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdgq.so")

OK = 0
DIM_AUTO, DIM_CHANNEL, DIM_PIXEL, DIM_BOTH = 0, 1, 2, 3
OUTLIER_KMEANS, OUTLIER_EXPLICIT = 0, 1
MODE_STATIC, MODE_DYNAMIC_TOKEN = 0, 1
CODES_U8, CODES_S8_CENTRED = 0, 1
SCALE_PER_PROMPT, SCALE_PER_PROMPT_HEAD, SCALE_PER_CALL = 0, 1, 2

EXPORTS = [
    "dgq_calibrate_groups", "dgq_groups_from_host", "dgq_groups_destroy", "dgq_groups_info",
    "dgq_groups_export", "dgq_quantize_act", "dgq_weight_prepare", "dgq_weight_from_codes",
    "dgq_weight_destroy", "dgq_weight_export", "dgq_linear", "dgq_linear_workspace_bytes", "dgq_cross_attn_logq", "dgq_cross_attn_logq_qv", "dgq_self_attn_logq",
    "dgq_cross_attn_workspace_bytes", "dgq_cross_attn_logq_noalloc", "dgq_selftest_wait_timeout", "dgq_device_status", "dgq_status_string", "dgq_launch_count",
]


class CalibConfig(C.Structure):
    _fields_ = [("act_bits", C.c_int), ("n_groups", C.c_int), ("dim_select", C.c_int),
                ("outlier_mode", C.c_int), ("outlier_tau", C.c_float), ("n_timesteps", C.c_int),
                ("rows_per_sample", C.c_int)]


class ConvDesc(C.Structure):
    _fields_ = [("n", C.c_int), ("h", C.c_int), ("w", C.c_int), ("c", C.c_int)]


class DgqError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2501_04304_b200.build`")
        _lib = C.CDLL(LIB_PATH)
        _lib.dgq_status_string.restype = C.c_char_p
        _lib.dgq_launch_count.restype = C.c_uint64
    return _lib


def status_string(s: int) -> str:
    return lib().dgq_status_string(C.c_int(s)).decode()


def _check(st, what):
    if st != OK:
        raise DgqError(st, what)


def _ptr(t):
    if t is None:
        return C.c_void_p(None)
    if isinstance(t, torch.Tensor):
        return C.c_void_p(t.data_ptr())
    if isinstance(t, np.ndarray):
        return C.c_void_p(t.ctypes.data)
    raise TypeError(type(t))


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def launch_count() -> int:
    return int(lib().dgq_launch_count())


def device_status() -> int:
    v = C.c_int(0)
    _check(lib().dgq_device_status(C.byref(v)), "dgq_device_status")
    return v.value


def selftest_wait_timeout(max_polls: int, stream=None):
    """dgq_selftest_wait_timeout: a kernel whose only wait runs out after `max_polls` polls."""
    _check(lib().dgq_selftest_wait_timeout(C.c_uint32(max_polls), _stream(stream)), "dgq_selftest_wait_timeout")


class Groups:
    """Owns a dgq_groups handle."""

    def __init__(self, handle):
        self.h = handle
        self._info()

    def _info(self):
        v = [C.c_int() for _ in range(8)]
        dc, dp = C.c_double(), C.c_double()
        _check(lib().dgq_groups_info(self.h, *[C.byref(x) for x in v], C.byref(dc), C.byref(dp)), "dgq_groups_info")
        (self.C, self.P, self.K_pad, self.G, self.R, self.T, self.dim, self.bits) = [x.value for x in v]
        self.D_channel, self.D_pixel = dc.value, dp.value

    def export(self):
        perm = np.empty(self.K_pad, np.int32)
        col_group = np.empty(self.C, np.int32)
        group_off = np.empty(self.G + 1, np.int32)
        row_group = np.empty(self.P, np.int32)
        scale = np.empty(self.T * self.R * self.G, np.float32)
        zp = np.empty(self.T * self.R * self.G, np.int32)
        _check(lib().dgq_groups_export(self.h, _ptr(perm), _ptr(col_group), _ptr(group_off), _ptr(row_group),
                                       _ptr(scale), _ptr(zp)), "dgq_groups_export")
        return dict(perm=perm, col_group=col_group, group_off=group_off, row_group=row_group,
                    scale=scale.reshape(self.T, self.R, self.G), zp=zp.reshape(self.T, self.R, self.G))

    def close(self):
        if self.h:
            lib().dgq_groups_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def calibrate_groups(X_cal, rows_per_sample, act_bits=8, n_groups=8, dim_select=DIM_AUTO,
                     outlier_mode=OUTLIER_KMEANS, outlier_tau=5.0, n_timesteps=1, timestep=0,
                     groups: Groups | None = None, stream=None) -> Groups:
    """dgq_calibrate_groups: X_cal is a CUDA fp16 [n_rows, C] tensor."""
    assert X_cal.is_cuda and X_cal.dtype == torch.float16 and X_cal.dim() == 2 and X_cal.stride(1) == 1
    cfg = CalibConfig(act_bits, n_groups, dim_select, outlier_mode, outlier_tau, n_timesteps, rows_per_sample)
    h = C.c_void_p(groups.h.value if groups is not None else None)
    st = lib().dgq_calibrate_groups(C.byref(cfg), _ptr(X_cal), C.c_int64(X_cal.shape[0]), C.c_int(X_cal.shape[1]),
                                    C.c_int64(X_cal.stride(0)), C.c_int(timestep), C.byref(h), _stream(stream))
    _check(st, "dgq_calibrate_groups")
    if groups is not None:
        groups._info()
        return groups
    return Groups(h)


def groups_from_host(C_, P, act_bits, col_group, row_group, scale, zp) -> Groups:
    """dgq_groups_from_host: scale, zp are [T, R, G] numpy arrays."""
    scale = np.ascontiguousarray(scale, np.float32)
    zp = np.ascontiguousarray(zp, np.int32)
    T, R, G = scale.shape
    cg = np.ascontiguousarray(col_group, np.int32)
    rg = np.ascontiguousarray(row_group, np.int32)
    h = C.c_void_p(None)
    st = lib().dgq_groups_from_host(C.c_int(C_), C.c_int(P), C.c_int(act_bits), C.c_int(G), C.c_int(R), C.c_int(T),
                                    _ptr(cg), _ptr(rg), _ptr(scale), _ptr(zp), C.byref(h))
    _check(st, "dgq_groups_from_host")
    return Groups(h)


def quantize_act(groups: Groups, X, timestep=0, mode=MODE_STATIC, layout=CODES_U8, out=None, stream=None):
    """dgq_quantize_act.  Returns (Xq uint8 [M, K_pad], dyn_scale or None, dyn_zp or None)."""
    assert X.is_cuda and X.dtype == torch.float16 and X.dim() == 2 and X.stride(1) == 1
    M = X.shape[0]
    Xq = out if out is not None else torch.empty((M, groups.K_pad), dtype=torch.uint8, device=X.device)
    ds = dz = None
    if mode == MODE_DYNAMIC_TOKEN:
        ds = torch.empty((M, groups.G), dtype=torch.float32, device=X.device)
        dz = torch.empty((M, groups.G), dtype=torch.int32, device=X.device)
    st = lib().dgq_quantize_act(groups.h, C.c_int(timestep), C.c_int(mode), C.c_int(layout), _ptr(X), C.c_int64(M),
                                C.c_int64(X.stride(0)), _ptr(Xq), _ptr(ds), _ptr(dz), _stream(stream))
    _check(st, "dgq_quantize_act")
    return Xq, ds, dz


def quantize_act_into(groups: Groups, X, Xq, ds, dz, timestep=0, mode=MODE_STATIC, layout=CODES_U8, stream=None):
    """dgq_quantize_act into caller-provided buffers (no allocation)."""
    st = lib().dgq_quantize_act(groups.h, C.c_int(timestep), C.c_int(mode), C.c_int(layout), _ptr(X),
                                C.c_int64(X.shape[0]), C.c_int64(X.stride(0)), _ptr(Xq), _ptr(ds), _ptr(dz),
                                _stream(stream))
    _check(st, "dgq_quantize_act")


class Weight:
    """Owns a dgq_weight handle."""

    def __init__(self, handle, N, K):
        self.h, self.N, self.K = handle, N, K

    def export(self):
        wq = np.empty((self.N, self.K), np.int8)
        sw = np.empty(self.N, np.float32)
        _check(lib().dgq_weight_export(self.h, _ptr(wq), _ptr(sw)), "dgq_weight_export")
        return wq, sw

    def close(self):
        if self.h:
            lib().dgq_weight_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _conv(conv):
    return C.byref(ConvDesc(*conv)) if conv is not None else C.c_void_p(None)


def weight_prepare(groups: Groups, W, w_bits=8, conv=None, stream=None) -> Weight:
    """dgq_weight_prepare: W is a CUDA fp16 [N, K] (or [N, 3, 3, C]) tensor; conv = (n, h, w, c) or None."""
    assert W.is_cuda and W.dtype == torch.float16 and W.is_contiguous()
    N = W.shape[0]
    K = W.numel() // N
    h = C.c_void_p(None)
    st = lib().dgq_weight_prepare(groups.h, _ptr(W), C.c_int(N), C.c_int(K), C.c_int(w_bits), _conv(conv),
                                  C.byref(h), _stream(stream))
    _check(st, "dgq_weight_prepare")
    return Weight(h, N, K)


def weight_from_codes(groups: Groups, wq, sw, w_bits=8, conv=None) -> Weight:
    wq = np.ascontiguousarray(wq, np.int8)
    sw = np.ascontiguousarray(sw, np.float32)
    N = wq.shape[0]
    K = wq.size // N
    h = C.c_void_p(None)
    st = lib().dgq_weight_from_codes(groups.h, _ptr(wq), _ptr(sw), C.c_int(N), C.c_int(K), C.c_int(w_bits),
                                     _conv(conv), C.byref(h))
    _check(st, "dgq_weight_from_codes")
    return Weight(h, N, K)


def linear_workspace_bytes(groups: Groups, weight: Weight, M: int) -> int:
    n = C.c_size_t(0)
    _check(lib().dgq_linear_workspace_bytes(groups.h, weight.h, C.c_int64(M), C.byref(n)), "dgq_linear_workspace_bytes")
    return n.value


def linear(groups: Groups, weight: Weight, Xq, timestep=0, mode=MODE_STATIC, layout=CODES_U8, dyn_scale=None,
           dyn_zp=None, bias=None, out=None, conv=None, workspace=None, stream=None):
    """dgq_linear.  Returns Y fp16 [M, N].  `workspace` (uint8 CUDA tensor) is only used for 4-bit
    weights; when it is None one of the size the library asks for is taken from torch, when it is
    False the call is made without one."""
    M = Xq.shape[0]
    Y = out if out is not None else torch.empty((M, weight.N), dtype=torch.float16, device=Xq.device)
    if workspace is False:
        workspace = None
    elif workspace is None:
        need = linear_workspace_bytes(groups, weight, M)
        workspace = torch.empty(need, dtype=torch.uint8, device=Xq.device) if need else None
    st = lib().dgq_linear(groups.h, weight.h, C.c_int(timestep), C.c_int(mode), C.c_int(layout), _ptr(Xq),
                          _ptr(dyn_scale), _ptr(dyn_zp), _ptr(bias), _ptr(Y), C.c_int64(M), C.c_int64(Y.stride(0)),
                          _conv(conv), _ptr(workspace), C.c_size_t(workspace.numel() if workspace is not None else 0),
                          _stream(stream))
    _check(st, "dgq_linear")
    return Y


def cross_attn_workspace_bytes(B, H, nq, nk, d) -> int:
    n = C.c_size_t(0)
    _check(lib().dgq_cross_attn_workspace_bytes(C.c_int(B), C.c_int(H), C.c_int(nq), C.c_int(nk), C.c_int(d),
                                                C.byref(n)), "dgq_cross_attn_workspace_bytes")
    return n.value


def cross_attn_logq(Q, K, V, score_bits=8, scale_gran=SCALE_PER_PROMPT, fixed_scale=None, out=None,
                    want_scale=False, want_codes=False, workspace=None, stream=None, v_bits=0):
    """dgq_cross_attn_logq (v_bits = 0) or dgq_cross_attn_logq_qv (quantized value operand, v_bits 2..8).
    Q [B, nq, H, d], K, V [B, nk, H, d] CUDA fp16.  Returns (O, scale, codes)."""
    B, nq, H, d = Q.shape
    nk = K.shape[1]
    assert Q.is_contiguous() and K.is_contiguous() and V.is_contiguous()
    O = out if out is not None else torch.empty_like(Q)
    n_scope = {SCALE_PER_PROMPT: B, SCALE_PER_PROMPT_HEAD: B * H, SCALE_PER_CALL: 1}[scale_gran]
    scale = torch.empty(n_scope, dtype=torch.float32, device=Q.device) if want_scale else None
    codes = torch.empty((B, H, nq, nk - 1), dtype=torch.uint8, device=Q.device) if want_codes else None
    need = cross_attn_workspace_bytes(B, H, nq, nk, d) if nk >= 2 else 256
    ws = workspace if workspace is not None else torch.empty(need, dtype=torch.uint8, device=Q.device)
    if v_bits:
        st = lib().dgq_cross_attn_logq_qv(_ptr(Q), _ptr(K), _ptr(V), C.c_int(B), C.c_int(H), C.c_int(nq), C.c_int(nk),
                                          C.c_int(d), C.c_int(score_bits), C.c_int(scale_gran), _ptr(fixed_scale),
                                          C.c_int(v_bits), _ptr(O), _ptr(scale), _ptr(codes), _ptr(ws),
                                          C.c_size_t(ws.numel()), _stream(stream))
        _check(st, "dgq_cross_attn_logq_qv")
        return O, scale, codes
    st = lib().dgq_cross_attn_logq(_ptr(Q), _ptr(K), _ptr(V), C.c_int(B), C.c_int(H), C.c_int(nq), C.c_int(nk),
                                   C.c_int(d), C.c_int(score_bits), C.c_int(scale_gran), _ptr(fixed_scale), _ptr(O),
                                   _ptr(scale), _ptr(codes), _ptr(ws), C.c_size_t(ws.numel()), _stream(stream))
    _check(st, "dgq_cross_attn_logq")
    return O, scale, codes


def self_attn_logq(Q, K, V, score_bits=8, fixed_scale=None, out=None, want_codes=False, stream=None):
    """dgq_self_attn_logq.  Q [B, nq, H, d], K, V [B, nk, H, d] CUDA fp16.  Returns (O, codes)."""
    B, nq, H, d = Q.shape
    nk = K.shape[1]
    assert Q.is_contiguous() and K.is_contiguous() and V.is_contiguous()
    O = out if out is not None else torch.empty_like(Q)
    codes = torch.empty((B, H, nq, nk), dtype=torch.uint8, device=Q.device) if want_codes else None
    st = lib().dgq_self_attn_logq(_ptr(Q), _ptr(K), _ptr(V), C.c_int(B), C.c_int(H), C.c_int(nq), C.c_int(nk),
                                  C.c_int(d), C.c_int(score_bits), _ptr(fixed_scale), _ptr(O), _ptr(codes),
                                  _stream(stream))
    _check(st, "dgq_self_attn_logq")
    return O, codes


NOALLOC_MAX_ROWS = 1 << 18
NOALLOC_MAX_HEADS = 256


def cross_attn_logq_noalloc(Q, K, V, O, score_bits=8, scale_gran=SCALE_PER_PROMPT, fixed_scale=None,
                            scale_out=None, codes_out=None, stream=None):
    """dgq_cross_attn_logq_noalloc: the same attention for callers that cannot provide a workspace.

    Every buffer, the output included, comes from the caller; neither this wrapper nor the
    library allocates.  The scratch is a fixed array inside the library, shared by all calls on a
    device, so calls that may overlap on the GPU must be serialised.  Limits: B * H * nq <=
    NOALLOC_MAX_ROWS and B * H <= NOALLOC_MAX_HEADS (status 4 beyond them).  The first call on a
    device should come before any stream capture.
    """
    B, nq, H, d = Q.shape
    nk = K.shape[1]
    st = lib().dgq_cross_attn_logq_noalloc(_ptr(Q), _ptr(K), _ptr(V), C.c_int(B), C.c_int(H), C.c_int(nq),
                                           C.c_int(nk), C.c_int(d), C.c_int(score_bits), C.c_int(scale_gran),
                                           _ptr(fixed_scale), _ptr(O), _ptr(scale_out), _ptr(codes_out),
                                           _stream(stream))
    _check(st, "dgq_cross_attn_logq_noalloc")
    return O
