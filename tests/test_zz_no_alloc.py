"""pevlm_query_attn_noalloc: the question attention for callers that cannot allocate device
memory (code in a memory-planned or real-time region, plug-ins without a memory pool).  It must
give what pevlm_query_attn gives with a caller workspace, call after call, although every call
shares one built-in scratch array that still holds the previous call's partials.

Collected last on purpose: a failure here leaves every other test already run.
"""
import numpy as np
import pytest

from paper_2506_19651_b200 import inputs
from helpers import LSE_TOL, O_TOL, bits_to_f64, to_bits, to_dev



def _case(S, B, N, Q, Hq, Hkv, d, seed):
    import torch
    from oracle import api as oracle
    from paper_2506_19651_b200 import binding as pb
    w = inputs.Workload("t", S, B, N, Q, Hq, Hkv, d, 1e6, True, seed)
    q, k, v = inputs.make_qkv(w)
    qr, kr = oracle.rope(q, w.theta), oracle.rope(k, w.theta)
    nv = w.n_video
    s = pb.make_shape(S, B, N, Q, Hq, Hkv, d, theta=w.theta)
    dq, dk, dv = to_dev(qr[nv:]), to_dev(kr), to_dev(v)
    mk = lambda: (torch.zeros((Q, Hq, d), dtype=torch.bfloat16, device="cuda"),
                  torch.zeros((Hq, Q), dtype=torch.float32, device="cuda"))
    o_ref, lse_ref = mk()
    ws = torch.zeros(pb.pevlm_workspace_bytes(s, pb.WS_QUERY), dtype=torch.uint8, device="cuda")
    pb.pevlm_query_attn(s, dq, dk, dv, o_ref, lse_ref, ws)
    o_new, lse_new = mk()
    pb.pevlm_query_attn_noalloc(s, dq, dk, dv, o_new, lse_new)
    torch.cuda.synchronize()
    assert pb.pevlm_read_status(ws)[0] == 0
    assert pb.pevlm_read_status(None) == (0, 0)      # the status header of the built-in array
    a, b = bits_to_f64(to_bits(o_new)), bits_to_f64(to_bits(o_ref))
    assert np.abs(a - b).max() <= O_TOL
    assert (lse_new - lse_ref).abs().max().item() <= LSE_TOL
    # and both agree with the oracle
    from oracle import api as oracle_api
    o_or, lse_or = oracle_api.attn_rows(oracle_api.make_shape(S, B, N, Q, Hq, Hkv, d), qr, kr, v, np.arange(nv, w.L))
    assert np.abs(a - o_or).max() <= O_TOL
    assert np.abs(lse_new.double().cpu().numpy().T - lse_or).max() <= LSE_TOL


@pytest.mark.gpu
def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    # two different shapes back to back: the second call finds the first call's partials in the array
    _case(200, 300, 3, 40, 4, 2, 128, seed=91)
    _case(64, 128, 4, 32, 4, 2, 64, seed=92)
    _case(200, 300, 3, 40, 4, 2, 128, seed=93)


def test_noalloc_rejects_shapes_beyond_the_builtin_array():
    # host-side check, made before any CUDA call: runs with or without a GPU
    import ctypes as C
    from paper_2506_19651_b200 import binding as pb
    big = pb.make_shape(1152, 1152, 63, 4096, 28, 4, 128, theta=1e6)
    assert pb.pevlm_workspace_bytes(big, pb.WS_QUERY) > pb.NOALLOC_SCRATCH_BYTES
    p16 = C.c_void_p(4096)
    rc = pb.lib().pevlm_query_attn_noalloc(C.byref(big), p16, p16, p16, p16, None, None)
    assert rc == pb.PEVLM_EWORKSPACE
    assert b"scratch bytes" in pb.lib().pevlm_last_cuda_error()
