"""GPU parity of the deferred index build (hdt_build_index returns once its work is queued; the
first call that needs the counts waits; hdt_attn_fwd on a bf16 index still in flight queues its
looping stage-0 kernel before that wait, with the counts read on the device): the same index, the
same attention results and the same errors as the waiting build, the errors only later."""
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


def batches():
    rng = np.random.default_rng(77)
    docs = gen.small_random_batch(210, n_seqs=4, max_len=500, K=(0, 40))
    ragged = gen.pack([gen.layout([[300, 2], [1, 131, 0]]), gen.layout([[7] * 40]),
                       (np.array([0], np.int8), np.array([-1], np.int32)),
                       (np.array([-1, -1, -1], np.int8), np.array([-1, -1, -1], np.int32)),
                       (np.zeros(0, np.int8), np.zeros(0, np.int32)),
                       gen.fit(*gen.layout([[5, 6], [7]]), 64, pad=True)])
    flat = gen.pack([(np.array([0], np.int8), np.array([-1], np.int32)) for _ in range(5)])     # one stage only
    trees = gen.pack([gen.layout_tree(gen.random_tree(rng, int(rng.integers(2, 6)), 5, p_leaf=0.4)) for _ in range(8)])
    return [("documents", docs), ("ragged", ragged), ("single tokens", flat), ("trees", trees)]


def attn_ws(P, b, H, d, dtype, bwd):
    """A workspace sized from a waiting build of the same batch (what a caller that wants the early
    launch has to provide: the size query itself would wait)."""
    idx = P.hdt_build_index(*dev_struct(b), max_stages=8)
    n = P.hdt_attn_workspace_bytes(idx, H, d, torch.bfloat16 if dtype == "bf16" else torch.float32, bwd)
    return torch.empty(max(n, 256), dtype=torch.uint8, device="cuda")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("d", [64, 128])
def test_deferred_matches_oracle(P, dtype, d):
    H = 2
    for i, (name, b) in enumerate(batches()):
        t = gen.make_tensors(300 + i, b.total_tokens, H, d, dtype)
        q, k, v, do = (dev_tensor(t[n], dtype) for n in ("q", "k", "v", "do"))
        o_r, lse_r = oracle.forward(b.level, b.parent, b.cu_seqlens, t["q"], t["k"], t["v"])
        dq_r, dk_r, dv_r = oracle.backward(b.level, b.parent, b.cu_seqlens, t["q"], t["k"], t["v"], t["do"])
        for own_ws in (True, False):
            ws_f = attn_ws(P, b, H, d, dtype, 0) if own_ws else None
            ws_b = attn_ws(P, b, H, d, dtype, 1) if own_ws else None
            idx = P.hdt_build_index(*dev_struct(b), max_stages=8, deferred=True)
            o, lse = P.hdt_attn_fwd(idx, q, k, v, workspace=ws_f)
            dq, dk, dv = P.hdt_attn_bwd(idx, q, k, v, o, lse, do, workspace=ws_b)
            check_close(host(o), o_r, dtype, f"{name} O")
            check_close(host(lse), lse_r, "f32" if dtype == "f32" else "bf16", f"{name} LSE")
            check_close(host(dq), dq_r, dtype, f"{name} dQ")
            check_close(host(dk), dk_r, dtype, f"{name} dK")
            check_close(host(dv), dv_r, dtype, f"{name} dV")
            P.hdt_device_status()


def test_deferred_index_is_bit_exact(P):
    for _, b in batches():
        want = ix.build(b.level, b.parent, b.cu_seqlens)
        idx = P.hdt_build_index(*dev_struct(b), max_stages=8, deferred=True)
        assert idx.nnz == want.nnz and idx.visited == want.visited and idx.n_stages == len(want.stages)
        for s, st in enumerate(want.stages):
            got = idx.export(s)
            for key in ("tok", "rng", "up", "blocks", "queue"):
                assert np.array_equal(got[key], getattr(st, key)), (s, key)


def test_deferred_same_result_as_waiting_build_repeated(P):
    """The early kernel and the kernels the host launches after its wait write the same bytes as the
    waiting path, call after call (graph replay of the build included)."""
    b = batches()[0][1]
    H, d = 3, 64
    t = gen.make_tensors(9, b.total_tokens, H, d, "bf16")
    q, k, v = (dev_tensor(t[n], "bf16") for n in ("q", "k", "v"))
    ws = attn_ws(P, b, H, d, "bf16", 0)
    st = dev_struct(b)
    o0, lse0 = P.hdt_attn_fwd(P.hdt_build_index(*st, max_stages=8), q, k, v, workspace=ws)
    o0, lse0 = o0.clone(), lse0.clone()
    for _ in range(5):
        idx = P.hdt_build_index(*st, max_stages=8, deferred=True)
        o, lse = P.hdt_attn_fwd(idx, q, k, v, workspace=ws)
        assert torch.equal(o, o0) and torch.equal(lse, lse0)


def test_deferred_errors_come_from_the_first_use(P):
    lv, pa = gen.layout([[2, 1], [1]])
    bad = pa.copy()
    bad[3] = 5                                              # parent after the token
    args = (torch.from_numpy(np.asarray(lv, np.int8)).cuda(), torch.from_numpy(np.asarray(bad, np.int32)).cuda(),
            torch.from_numpy(np.array([0, 10], np.int32)).cuda())
    with pytest.raises(P.HdtError) as e:
        P.hdt_build_index(*args)                            # the waiting build reports it itself
    assert e.value.code == -2
    idx = P.hdt_build_index(*args, deferred=True)           # the deferred one returns ...
    q = torch.zeros((10, 1, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.HdtError) as e:                    # ... and the first use reports it
        P.hdt_attn_fwd(idx, q, q, q, workspace=torch.empty(1 << 16, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -2
    with pytest.raises(P.HdtError) as e:                    # every later use too
        idx.n_stages
    assert e.value.code == -2
    # deeper than max_stages
    deep = gen.layout_tree([[[[[[]]]]]])
    idx = P.hdt_build_index(torch.from_numpy(deep[0]).cuda(), torch.from_numpy(deep[1]).cuda(),
                            torch.from_numpy(np.array([0, len(deep[0])], np.int32)).cuda(), max_stages=2, deferred=True)
    with pytest.raises(P.HdtError) as e:
        idx.nnz
    assert e.value.code == -2
    # the context is still usable afterwards
    b = batches()[0][1]
    assert P.hdt_build_index(*dev_struct(b), deferred=True).nnz == ix.build(b.level, b.parent, b.cu_seqlens).nnz
    P.hdt_device_status()


def test_deferred_workspace_too_small(P):
    """The early kernel finds a workspace that cannot hold stage 1's partial results on the device and
    does nothing; the host finds the same after its wait and reports it."""
    b = batches()[0][1]
    H, d = 2, 64
    t = gen.make_tensors(5, b.total_tokens, H, d, "bf16")
    q, k, v = (dev_tensor(t[n], "bf16") for n in ("q", "k", "v"))
    idx = P.hdt_build_index(*dev_struct(b), max_stages=8, deferred=True)
    with pytest.raises(P.HdtError) as e:
        P.hdt_attn_fwd(idx, q, k, v, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -4
    o, lse = P.hdt_attn_fwd(idx, q, k, v)                   # the index itself is fine
    o_r, _ = oracle.forward(b.level, b.parent, b.cu_seqlens, t["q"], t["k"], t["v"])
    check_close(host(o), o_r, "bf16", "O")
    P.hdt_device_status()


def test_deferred_full_size_sampled(P):
    """The configuration the benchmark times (deferred build, caller workspaces), sampled rows and keys."""
    c = 3
    cfg = gen.CONFIGS[c]
    b = gen.make_hierarchy(c)
    T, H, d = b.total_tokens, cfg.heads, cfg.head_dim
    t = gen.make_tensors(cfg.tensor_seed, T, H, d, cfg.dtype)
    q, k, v, do = (dev_tensor(t[n], cfg.dtype) for n in ("q", "k", "v", "do"))
    ws_f, ws_b = attn_ws(P, b, H, d, cfg.dtype, 0), attn_ws(P, b, H, d, cfg.dtype, 1)
    idx = P.hdt_build_index(*dev_struct(b), max_stages=4, deferred=True)
    o, lse = P.hdt_attn_fwd(idx, q, k, v, workspace=ws_f)
    dq, dk, dv = P.hdt_attn_bwd(idx, q, k, v, o, lse, do, workspace=ws_b)
    rng = np.random.default_rng(c)
    anchors = np.flatnonzero((b.level >= 0) & (b.level < 3))
    sample = np.unique(np.concatenate([rng.choice(T, 40, replace=False), rng.choice(anchors, 12, replace=False),
                                       b.cu_seqlens[:-1], b.cu_seqlens[1:] - 1])).astype(np.int32)
    s64 = sample.astype(np.int64)
    o_r, lse_r, dq_r = oracle.rows(b.level, b.parent, b.cu_seqlens, t["q"], t["k"], t["v"], sample, do=t["do"])
    dk_r, dv_r = oracle.cols(b.level, b.parent, b.cu_seqlens, t["q"], t["k"], t["v"], t["do"], sample)
    check_close(host(o[s64]), o_r, cfg.dtype, "O")
    check_close(host(lse[:, s64]).T, lse_r, cfg.dtype, "LSE")
    check_close(host(dq[s64]), dq_r, cfg.dtype, "dQ")
    check_close(host(dk[s64]), dk_r, cfg.dtype, "dK")
    check_close(host(dv[s64]), dv_r, cfg.dtype, "dV")
    for x in (o, dq, dk, dv):
        assert torch.isfinite(x.float()).all()
    P.hdt_device_status()


def test_many_steps_no_expired_wait_and_same_bytes(P):
    """800 steps of the benchmark's configuration (deferred build, caller workspaces, forward and backward,
    L2 flushed in between): no bounded wait of a kernel runs out (a thread of a looping kernel that
    reaches its wait on a barrier after the barrier has been re-armed twice waits for a phase that has
    passed; seen once in fifteen and once in a thousand steps while the looping forward was rebuilt)
    and every step writes the same bytes."""
    c = 3
    cfg = gen.CONFIGS[c]
    b = gen.make_hierarchy(c)
    T, H, d = b.total_tokens, cfg.heads, cfg.head_dim
    t = gen.make_tensors(cfg.tensor_seed, T, H, d, cfg.dtype)
    q, k, v, do = (dev_tensor(t[n], cfg.dtype) for n in ("q", "k", "v", "do"))
    ws_f, ws_b = attn_ws(P, b, H, d, cfg.dtype, 0), attn_ws(P, b, H, d, cfg.dtype, 1)
    st = dev_struct(b)
    flush = torch.empty(192 << 20, dtype=torch.uint8, device="cuda")
    first = None
    for i in range(800):
        flush.zero_()
        idx = P.hdt_build_index(*st, max_stages=4, deferred=True)
        o, lse = P.hdt_attn_fwd(idx, q, k, v, workspace=ws_f)
        dq, dk, dv = P.hdt_attn_bwd(idx, q, k, v, o, lse, do, workspace=ws_b)
        if i % 100 == 0:
            P.hdt_device_status()
            if first is None:
                first = [x.clone() for x in (o, lse, dq, dk, dv)]
            else:
                for x, y in zip((o, lse, dq, dk, dv), first):
                    assert torch.equal(x, y)
    P.hdt_device_status()


def test_many_steps_split_families_no_expired_wait(P):
    """400 forward and backward steps of the skewed configuration (families of up to nine key chunks:
    the multi-chunk forward and the persistent backward with their tile rings and MMA barriers), L2
    flushed in between: no bounded wait runs out and the forward writes the same bytes every step."""
    c = 5
    cfg = gen.CONFIGS[c]
    b = gen.make_hierarchy(c)
    T, H, d = b.total_tokens, cfg.heads, cfg.head_dim
    t = gen.make_tensors(cfg.tensor_seed, T, H, d, cfg.dtype)
    q, k, v, do = (dev_tensor(t[n], cfg.dtype) for n in ("q", "k", "v", "do"))
    st = dev_struct(b)
    flush = torch.empty(192 << 20, dtype=torch.uint8, device="cuda")
    first = None
    for i in range(400):
        flush.zero_()
        idx = P.hdt_build_index(*st, max_stages=4, deferred=True)
        o, lse = P.hdt_attn_fwd(idx, q, k, v)
        P.hdt_attn_bwd(idx, q, k, v, o, lse, do)
        if i % 100 == 0:
            P.hdt_device_status()
            if first is None:
                first = [x.clone() for x in (o, lse)]
            else:
                for x, y in zip((o, lse), first):
                    assert torch.equal(x, y)
    P.hdt_device_status()
