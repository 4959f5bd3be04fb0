"""The workspace-free cross-attention entry point against the ordinary one.

Some callers cannot hand the library a workspace because they cannot allocate device memory at
the point of the call (a plugin that only receives its input and output buffers, a loop that must
stay clear of the allocator).  For them the library keeps a fixed scratch array of its own.  This
test calls that entry point through the C ABI twice in a row, with different inputs, so that the
second call starts on the first call's leftovers, and checks each result against the ordinary
entry point.  It sits in a file that pytest collects last.
"""
import numpy as np
import pytest

from paper_2501_04304_b200 import synth
from dgq_testlib import gpu, to_dev

pytestmark = pytest.mark.gpu


def test_noalloc_matches_workspace_entry_point_twice():
    torch, b = gpu()
    for call, (seed, B, H, nq, bits) in enumerate([(21, 2, 8, 300, 8), (22, 1, 4, 515, 4)]):
        Q, K, V = [to_dev(torch, x) for x in synth.attention_inputs(seed, B, H, nq, 77, 40)]
        O_ref, s_ref, c_ref = b.cross_attn_logq(Q, K, V, bits, want_scale=True, want_codes=True)
        O = torch.empty_like(Q)
        s = torch.empty_like(s_ref)
        c = torch.empty_like(c_ref)
        if call == 1:
            # the entry point itself takes no device memory: neither the driver's free-memory figure nor
            # torch's allocator moves across the call (every buffer above was made before it)
            torch.cuda.synchronize()
            free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        b.cross_attn_logq_noalloc(Q, K, V, O, bits, scale_out=s, codes_out=c)
        if call == 1:
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
        assert b.device_status() == 0
        ref = O_ref.float().cpu().numpy()
        got = O.float().cpu().numpy()
        assert np.max(np.abs(got - ref)) <= 1e-3 * np.max(np.abs(ref)), f"call {call}"
        assert torch.equal(c, c_ref) and torch.equal(s, s_ref), f"call {call}"


def test_noalloc_rejects_oversized_problem():
    torch, b = gpu()
    Q, K, V = [to_dev(torch, x) for x in synth.attention_inputs(23, 1, 1, 16, 4, 40, ctx_dim=16)]
    O = torch.empty_like(Q)
    lib = b.lib()
    import ctypes as C
    # B * H * nq beyond the built-in scratch: refused before anything is launched
    st = lib.dgq_cross_attn_logq_noalloc(C.c_void_p(Q.data_ptr()), C.c_void_p(K.data_ptr()), C.c_void_p(V.data_ptr()),
                                         C.c_int(64), C.c_int(8), C.c_int(4096), C.c_int(4), C.c_int(40), C.c_int(8),
                                         C.c_int(0), None, C.c_void_p(O.data_ptr()), None, None, None)
    assert st == 4
    st = lib.dgq_cross_attn_logq_noalloc(C.c_void_p(Q.data_ptr()), C.c_void_p(K.data_ptr()), C.c_void_p(V.data_ptr()),
                                         C.c_int(300), C.c_int(1), C.c_int(1), C.c_int(4), C.c_int(40), C.c_int(8),
                                         C.c_int(0), None, C.c_void_p(O.data_ptr()), None, None, None)
    assert st == 4
    # few heads but too many rows for the row statistics
    st = lib.dgq_cross_attn_logq_noalloc(C.c_void_p(Q.data_ptr()), C.c_void_p(K.data_ptr()), C.c_void_p(V.data_ptr()),
                                         C.c_int(1), C.c_int(8), C.c_int(40000), C.c_int(4), C.c_int(40), C.c_int(8),
                                         C.c_int(0), None, C.c_void_p(O.data_ptr()), None, None, None)
    assert st == 4
    # an ordinary argument error on an oversized problem is reported as what it is (nk < 2: invalid argument)
    st = lib.dgq_cross_attn_logq_noalloc(C.c_void_p(Q.data_ptr()), C.c_void_p(K.data_ptr()), C.c_void_p(V.data_ptr()),
                                         C.c_int(64), C.c_int(8), C.c_int(4096), C.c_int(1), C.c_int(40), C.c_int(8),
                                         C.c_int(0), None, C.c_void_p(O.data_ptr()), None, None, None)
    assert st == 1


def test_noalloc_accepts_the_largest_problem():
    """B * H = 256 heads and B * H * nq = 2^18 rows are the stated limits: the call must fit its scratch
    (row statistics plus one partial maximum per block of query rows) and agree with the ordinary entry point."""
    torch, b = gpu()
    B, H, nq = 32, 8, 1024
    Q, K, V = [to_dev(torch, x) for x in synth.attention_inputs(25, B, H, nq, 77, 40)]
    O_ref, s_ref, _ = b.cross_attn_logq(Q, K, V, 8, want_scale=True)
    O = torch.empty_like(Q)
    s = torch.empty_like(s_ref)
    b.cross_attn_logq_noalloc(Q, K, V, O, 8, scale_out=s)
    assert b.device_status() == 0
    assert torch.equal(s, s_ref) and torch.equal(O, O_ref)
