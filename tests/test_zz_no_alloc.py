"""hdt_attn_fwd_static: the forward pass for callers that cannot allocate device memory.

Its scratch is a fixed array inside the library, shared by all calls, so the test checks two calls
in a row (the second one starts from whatever the first left in the array) against the ordinary
hdt_attn_fwd, which uses a caller workspace, and against the fp64 oracle.  Before them a call with
NaN inputs fills the part of the array these batches use with NaN, so a read of a stale entry would
show.  This file sorts last on purpose: a run that stops at the first failure has then already run
every other test."""
import numpy as np
import pytest
import torch

import gen
import oracle
from gpu_util import check_close, dev_struct, dev_tensor, host

pytestmark = pytest.mark.gpu


def _case(P, b, H, d, dtype, seed):
    t = gen.make_tensors(seed, b.total_tokens, H, d, dtype)
    idx = P.hdt_build_index(*dev_struct(b), max_stages=8)
    q, k, v = (dev_tensor(t[n], dtype) for n in ("q", "k", "v"))
    return b, t, idx, q, k, v


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_static_scratch_forward_matches_workspace_forward_twice(dtype):
    import paper_2407_08330_b200 as P
    # different batches back to back: each call finds the previous call's leftovers; the second is
    # padded (PAD tails: EMPTY row blocks), the third has another head_dim
    cases = [_case(P, gen.small_random_batch(71, n_seqs=4, max_len=500, K=(0, 40)), 3, 64, dtype, 1),
             _case(P, gen.small_random_batch(72, n_seqs=3, pad_to=700, max_len=420, K=(0, 30)), 2, 64, dtype, 3),
             _case(P, gen.make_hierarchy(1), 2, 128, dtype, 2)]
    # poison: the largest batch once with NaN queries, so that every partial result in the array is NaN
    _, _, idx0, q0, k0, v0 = cases[0]
    P.hdt_attn_fwd_static(idx0, torch.full_like(q0, float("nan")), k0, v0)
    torch.cuda.synchronize()
    for b, t, idx, q, k, v in cases:
        want_o, want_lse = P.hdt_attn_fwd(idx, q, k, v)
        out = torch.empty_like(q)
        lse = torch.empty((q.shape[1], q.shape[0]), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info()[0]                    # the driver's count: sees any cudaMalloc
        before = torch.cuda.memory_stats()["allocation.all.allocated"]   # torch's allocator, cumulative
        got_o, got_lse = P.hdt_attn_fwd_static(idx, q, k, v, out=out, lse=lse)
        torch.cuda.synchronize()
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == before
        assert torch.cuda.mem_get_info()[0] >= free0            # nothing was allocated on the device
        P.hdt_device_status()
        tol = 2e-2 if dtype == "bf16" else 1e-4
        assert float((got_o.float() - want_o.float()).abs().max()) <= tol
        fin = torch.isfinite(want_lse)
        assert torch.equal(torch.isfinite(got_lse), fin)
        assert float((got_lse[fin] - want_lse[fin]).abs().max()) <= tol
        o_r, lse_r = oracle.forward(b.level, b.parent, b.cu_seqlens, t["q"], t["k"], t["v"])
        check_close(host(got_o), o_r, dtype, "O (static scratch)")
        check_close(host(got_lse), lse_r, dtype, "LSE (static scratch)")


def test_static_scratch_rejects_batches_beyond_its_size():
    import paper_2407_08330_b200 as P
    rng = np.random.default_rng(9)
    b = gen.pack([gen.gen_fill(rng, 6000, (4, 24), (3, 20), (5, 20)) for _ in range(4)])
    H, d = 32, 128
    idx = P.hdt_build_index(*dev_struct(b))
    need = P.hdt_attn_workspace_bytes(idx, H, d, torch.bfloat16, 0)
    assert need > P.hdt_attn_fwd_static_max_bytes()
    q = torch.zeros((b.total_tokens, H, d), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.HdtError) as e:
        P.hdt_attn_fwd_static(idx, q, q, q)
    assert e.value.code == -4 and "scratch" in str(e.value)
    # the ordinary entry point still serves that batch
    o, lse = P.hdt_attn_fwd(idx, q, q, q)
    assert torch.isfinite(o.float()).all()
