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
