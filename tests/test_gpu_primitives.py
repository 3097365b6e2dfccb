"""tcgen05 / TMA primitives: one-CTA GEMM through the test hook against a plain matmul, for every
operand-major combination the attention kernels use."""
import ctypes as C

import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("a_mn", [0, 1])
@pytest.mark.parametrize("b_mn", [0, 1])
@pytest.mark.parametrize("N,K", [(128, 64), (64, 128), (16, 16), (48, 112), (128, 128)])
def test_debug_gemm(a_mn, b_mn, N, K):
    import paper_2407_08330_b200 as P
    L = P.lib()
    torch.manual_seed(N * 1000 + K + 10 * a_mn + b_mn)
    A = torch.randn(128, K, device="cuda").to(torch.bfloat16)
    B = torch.randn(N, K, device="cuda").to(torch.bfloat16)
    a = A.t().contiguous() if a_mn else A.contiguous()
    b = B.t().contiguous() if b_mn else B.contiguous()
    c = torch.full((128, N), float("nan"), device="cuda")
    L.hdt_debug_gemm.restype = C.c_int
    rc = L.hdt_debug_gemm(C.c_void_p(a.data_ptr()), C.c_void_p(b.data_ptr()), C.c_void_p(c.data_ptr()),
                          C.c_int32(N), C.c_int32(K), C.c_int32(a_mn), C.c_int32(b_mn),
                          C.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == 0, L.hdt_last_error()
    want = A.float() @ B.float().t()
    assert torch.allclose(c, want, atol=1e-3, rtol=1e-3), float((c - want).abs().max())


def test_bounded_wait_gives_up_reports_and_leaves_the_library_usable():
    """The failure path of the kernels' bounded waits, run on purpose and safely: one CTA waits on a
    barrier that nothing was ever issued to complete (no copy, no MMA in flight), with a limit of 1e5
    cycles.  The wait must give up, the status word must carry HDT_ERR_TIMEOUT with the kernel and
    the site, TMEM must have been released (the next tensor-core kernels get their columns), and
    the next ordinary calls must pass."""
    import numpy as np

    import gen
    import oracle
    import paper_2407_08330_b200 as P
    from gpu_util import check_close, dev_struct, dev_tensor, host
    L = P.lib()
    P.hdt_device_status()                         # nothing pending from earlier tests
    L.hdt_debug_wait_timeout.restype = C.c_int
    early = C.c_int32(-1)
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    rc = L.hdt_debug_wait_timeout(C.c_int64(100000), C.byref(early), stream)
    assert rc == -6, (rc, L.hdt_last_error())                          # HDT_ERR_TIMEOUT
    msg = L.hdt_last_error().decode()
    assert "kernel 15" in msg and "wait 1" in msg, msg
    assert 0 <= early.value <= 128
    P.hdt_device_status()                         # reported once, then cleared
    # the library works as before: a bf16 forward + backward on the tensor-core kernels against the oracle
    b = gen.small_random_batch(91, n_seqs=3, max_len=400, K=(0, 40))
    t = gen.make_tensors(9, b.total_tokens, 2, 64, "bf16")
    idx = P.hdt_build_index(*dev_struct(b))
    q, k, v, do = (dev_tensor(t[n], "bf16") for n in ("q", "k", "v", "do"))
    o, lse = P.hdt_attn_fwd(idx, q, k, v)
    dq, dk, dv = P.hdt_attn_bwd(idx, q, k, v, o, lse, do)
    P.hdt_device_status()
    o_r, _ = oracle.forward(b.level, b.parent, b.cu_seqlens, t["q"], t["k"], t["v"])
    dq_r, _, _ = oracle.backward(b.level, b.parent, b.cu_seqlens, t["q"], t["k"], t["v"], t["do"])
    check_close(host(o), o_r, "bf16", "O after a recorded timeout")
    check_close(host(dq), dq_r, "bf16", "dQ after a recorded timeout")
    # a limit outside the accepted range is refused on the host
    assert L.hdt_debug_wait_timeout(C.c_int64(10), None, stream) == -1
