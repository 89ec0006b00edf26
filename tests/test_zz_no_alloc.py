"""dsq_gemm_static_ws: the GEMM entry point for callers that cannot allocate
device memory (hosts that own the whole memory pool, plug-ins, real-time
loops where cudaMalloc is off limits).  It must give exactly what dsq_gemm
gives, call after call, although its scratch is one static array that keeps
whatever the previous call left in it.

Collected last on purpose: a run that stops at the first failure has then
already been through every other test."""
import ctypes as C

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from oracle import native
import dsq_inputs
from gpu_util import T, N


def test_static_workspace_gemm_matches_dsq_gemm_twice_in_a_row():
    import paper_1908_05033_b200 as dsq
    lib = dsq.lib
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    ws = dsq.new_workspace()
    # two different problems back to back: the second call meets the first
    # call's leftovers in the shared scratch
    for (M, Nn, K, bits) in [(300, 257, 1000, 4), (515, 130, 771, 2)]:
        A, B, rs = dsq_inputs.gemm_case(M, Nn, K, bits)
        Ap, Bp = dsq.dsq_pack_codes(T(A), bits), dsq.dsq_pack_codes(T(B), bits)
        rs_t = T(rs)
        C_ref, D_ref = dsq.dsq_gemm(Ap, Bp, M, Nn, K, bits, ws, row_scale=rs_t)
        assert dsq.dsq_workspace_status(ws) == 0
        # the caller owns inputs and outputs; the entry point gets raw pointers
        C_out = torch.full((M, Nn), -1, dtype=torch.int32, device="cuda")
        D_out = torch.full((M, Nn), float("nan"), dtype=torch.float32, device="cuda")
        st = lib.dsq_gemm_static_ws(
            C.c_void_p(Ap.data_ptr()), C.c_void_p(Bp.data_ptr()), M, Nn, K, bits,
            C.c_void_p(C_out.data_ptr()), C.c_void_p(rs_t.data_ptr()),
            C.c_void_p(D_out.data_ptr()), 1, stream)
        assert st == 0
        # integer results bit-exact, fp32 results bit-exact (one multiply),
        # the tolerance the GEMM parity tests use
        assert torch.equal(C_out, C_ref)
        assert torch.equal(D_out, D_ref)
        # ... and the oracle's (the same sizes are among the GEMM parity cases)
        C_cpu = native.gemm(A, B)
        assert np.array_equal(N(C_out), C_cpu)
        assert np.array_equal(N(D_out), native.gemm_dequant(C_cpu, rs))
        # enqueue-only form: returns at once, the caller synchronises
        C_out.fill_(-1)
        st = lib.dsq_gemm_static_ws(
            C.c_void_p(Ap.data_ptr()), C.c_void_p(Bp.data_ptr()), M, Nn, K, bits,
            C.c_void_p(C_out.data_ptr()), None, None, 0, stream)
        assert st == 0
        torch.cuda.synchronize()
        assert torch.equal(C_out, C_ref)
    # the documented limit is enforced before anything is launched
    st = lib.dsq_gemm_static_ws(C.c_void_p(Ap.data_ptr()), C.c_void_p(Bp.data_ptr()),
                                65537, 16, 16, 4, C.c_void_p(C_out.data_ptr()), None, None,
                                1, stream)
    assert st == -5
    # a rejected call leaves the stream and the outputs untouched
    C_out.fill_(7)
    st = lib.dsq_gemm_static_ws(None, C.c_void_p(Bp.data_ptr()), M, Nn, K, bits,
                                C.c_void_p(C_out.data_ptr()), None, None, 1, stream)
    assert st == -1
    st = lib.dsq_gemm_static_ws(C.c_void_p(Ap.data_ptr()), C.c_void_p(Bp.data_ptr()), M, Nn, K,
                                5, C.c_void_p(C_out.data_ptr()), None, None, 1, stream)
    assert st == -3
    torch.cuda.synchronize()
    assert bool((C_out == 7).all())
