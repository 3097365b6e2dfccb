"""GPU parity of the directed mask variants (child->parent, sibling<->sibling, parent->child groups
switched on and off) against the fp64 oracle: index totals bit-exact, forward and backward within
the fp32 / bf16 tolerances, on documents, deep expression trees and a ListOps-shaped batch."""
import numpy as np
import pytest
import torch

import gen
import oracle
from oracle import index_oracle as ix
from gpu_util import check_close, dev_struct, dev_tensor, host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P():
    import paper_2407_08330_b200 as P
    return P


def small_batches():
    rng = np.random.default_rng(31)
    docs = gen.small_random_batch(32, n_seqs=4, max_len=300, K=(0, 30))
    trees = gen.pack([gen.layout_tree(gen.listops_tree(rng, 8, 5, 120, 0.45)) for _ in range(6)])
    long_family = gen.pack([gen.layout([[150, 3], [2]])])      # a family longer than a row block
    return [("documents", docs), ("trees", trees), ("long family", long_family)]


@pytest.mark.parametrize("d", [6, 4, 0, 1, 2, 3, 5])
def test_index_totals_with_directions(P, d):
    for _, b in small_batches():
        want = ix.build(b.level, b.parent, b.cu_seqlens, directions=d)
        idx = P.hdt_build_index(*dev_struct(b), max_stages=12, directions=d)
        assert idx.nnz == want.nnz and idx.visited == want.visited and idx.n_stages == len(want.stages)
        for s, st in enumerate(want.stages):
            got = idx.export(s)
            assert np.array_equal(got["rng"], st.rng) and np.array_equal(got["blocks"], st.blocks)


def run(P, b, H, dim, dtype, d, seed):
    t = gen.make_tensors(seed, b.total_tokens, H, dim, dtype)
    # Without the sibling group an anchor collects the whole probability mass of its children and
    # gradients reach 20 and more, where the spacing of bf16 outputs alone (0.125) exceeds the
    # absolute tolerance: gradients may exceed the maximum by half a bf16 ulp of the expected value
    # (the rounding of the stored result), element by element; dO stays N(0,1).
    idx = P.hdt_build_index(*dev_struct(b), max_stages=12, directions=d)
    q, k, v, do = (dev_tensor(t[n], dtype) for n in ("q", "k", "v", "do"))
    o, lse = P.hdt_attn_fwd(idx, q, k, v)
    o_r, lse_r = oracle.forward(b.level, b.parent, b.cu_seqlens, t["q"], t["k"], t["v"], directions=d)
    check_close(host(o), o_r, dtype, "O")
    check_close(host(lse), lse_r, "f32" if dtype == "f32" else "bf16", "LSE")
    dq, dk, dv = P.hdt_attn_bwd(idx, q, k, v, o, lse, do)
    dq_r, dk_r, dv_r = oracle.backward(b.level, b.parent, b.cu_seqlens, t["q"], t["k"], t["v"], t["do"], directions=d)
    # (row_rel: the bf16 rounding of P and dS inside the kernels, 2^-9 relative per term, grows with them)
    check_close(host(dq), dq_r, dtype, "dQ", out_rounding=True, row_rel=2.0 ** -8)
    check_close(host(dk), dk_r, dtype, "dK", out_rounding=True, row_rel=2.0 ** -8)
    check_close(host(dv), dv_r, dtype, "dV", out_rounding=True, row_rel=2.0 ** -8)
    P.hdt_device_status()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d", [6, 4, 0, 3, 5])
def test_directed_attention_small(P, d, dtype):
    for i, (_, b) in enumerate(small_batches()):
        run(P, b, 2, 64, dtype, d, 40 + i)


def test_directed_attention_general_and_simt_paths_bf16(P):
    b = small_batches()[0][1]
    for opt in ({"no_overlap": 1}, {"no_persistent": 1}, {"force_simt": 1}):
        for k_, v_ in opt.items():
            P.hdt_set_option(k_, v_)
        try:
            run(P, b, 2, 128, "bf16", 6, 50)
        finally:
            for k_ in opt:
                P.hdt_set_option(k_, 0)


def test_listops_batch_sampled(P):
    """The ListOps-shaped batch (200 trees, depth up to 20) with operands not attending to their
    operators: sampled rows and keys against the oracle, properties at full size."""
    c, d = 7, 6
    cfg = gen.CONFIGS[c]
    b = gen.make_hierarchy(c)
    T, H, dim = b.total_tokens, cfg.heads, cfg.head_dim
    t = gen.make_tensors(cfg.tensor_seed, T, H, dim, cfg.dtype)
    idx = P.hdt_build_index(*dev_struct(b), max_stages=24, directions=d)
    assert idx.n_stages == 20
    q, k, v, do = (dev_tensor(t[n], cfg.dtype) for n in ("q", "k", "v", "do"))
    o, lse = P.hdt_attn_fwd(idx, q, k, v)
    dq, dk, dv = P.hdt_attn_bwd(idx, q, k, v, o, lse, do)
    P.hdt_device_status()
    rng = np.random.default_rng(c)
    sample = np.unique(np.concatenate([rng.choice(T, 64, replace=False), b.cu_seqlens[:4], b.cu_seqlens[1:5] - 1])).astype(np.int32)
    o_r, lse_r, dq_r = oracle.rows(b.level, b.parent, b.cu_seqlens, t["q"], t["k"], t["v"], sample, do=t["do"], directions=d)
    dk_r, dv_r = oracle.cols(b.level, b.parent, b.cu_seqlens, t["q"], t["k"], t["v"], t["do"], sample, directions=d)
    s64 = sample.astype(np.int64)
    check_close(host(o[s64]), o_r, cfg.dtype, "O")
    check_close(host(lse[:, s64]).T, lse_r, cfg.dtype, "LSE")
    check_close(host(dq[s64]), dq_r, cfg.dtype, "dQ")
    check_close(host(dk[s64]), dk_r, cfg.dtype, "dK")
    check_close(host(dv[s64]), dv_r, cfg.dtype, "dV")
    for x in (o, dq, dk, dv):
        assert torch.isfinite(x.float()).all()
    # without the child->parent group the root of every tree is attended by nobody but itself
    roots = torch.from_numpy(b.cu_seqlens[:-1].astype(np.int64)).cuda()
    p_self = torch.exp((q[roots].float() * k[roots].float()).sum(-1) / np.sqrt(dim) - lse[:, roots].T)
    assert torch.allclose(dv[roots].float(), p_self[..., None] * do[roots].float(), atol=2e-2)
