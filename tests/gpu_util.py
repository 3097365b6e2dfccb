"""Helpers for the GPU parity tests: move seeded inputs to the device, compare with the oracle."""
import numpy as np
import torch

import gen

TOL = {"bf16": dict(max=2e-2, mean=2e-3), "f32": dict(max=1e-4, mean=1e-4)}


def dev_struct(b):
    return (torch.from_numpy(b.level).cuda(), torch.from_numpy(b.parent).cuda(),
            torch.from_numpy(b.cu_seqlens).cuda())


def dev_tensor(x, dtype):
    t = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t   # values are bf16-representable: exact


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def half_ulp_bf16(x):
    """Half the spacing of the bf16 grid at |x| (8 significant bits): what storing x as bf16 can add
    to its error at most.  0 for x = 0."""
    ax = np.abs(np.asarray(x, np.float64))
    e = np.floor(np.log2(np.where(ax > 0, ax, 1.0)))
    return np.where(ax > 0, np.ldexp(1.0, (e - 8).astype(np.int64)), 0.0)


def check_close(got, want, dtype, what, out_rounding=False, row_rel=0.0):
    """Element-wise comparison against the oracle at the stated tolerances (max and mean absolute
    error: bf16 2e-2 / 2e-3, fp32 1e-4).
    out_rounding (bf16 results whose magnitude can pass 4, where the bf16 grid itself is coarser than
    the tolerance): every element may exceed the maximum by half a bf16 ulp of the expected value,
    i.e. by the rounding of the stored result, and the mean by the mean of a quarter ulp (the
    expected size of that rounding), so the kernel's own error is still held to the tolerance.
    row_rel (only for inputs outside the named configurations that make gradients of size 10 and
    more: a softmax scale of 0.2, directed masks without the sibling group): the bf16 kernels round P
    and dS to 8 significant bits before the tensor-core products, a relative error of 2^-9 per term
    that grows with the gradients; an element may additionally be off by row_rel times the largest
    expected magnitude in its (token, head) row."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    fin = np.isfinite(want)
    assert np.array_equal(np.isfinite(got), fin), f"{what}: finiteness differs"
    assert np.array_equal(got[~fin], want[~fin]), f"{what}: non-finite values differ"
    err = np.abs(got[fin] - want[fin])
    tol = TOL[dtype]
    bound = np.full(err.shape, tol["max"])
    mean_bound = tol["mean"]
    if out_rounding and dtype == "bf16":
        hu = half_ulp_bf16(want[fin])
        bound = bound + hu
        mean_bound += float(hu.mean()) / 2 if hu.size else 0.0
    if row_rel and dtype == "bf16" and want.ndim >= 2:
        rowmax = np.where(fin, np.abs(want), 0.0).max(axis=-1, keepdims=True)
        bound = bound + row_rel * np.broadcast_to(rowmax, want.shape)[fin]
    over = err - bound
    mx = float(err.max()) if err.size else 0.0
    mean = float(err.mean()) if err.size else 0.0
    worst = float(over.max()) if err.size else -1.0
    assert worst <= 0 and mean <= mean_bound, \
        f"{what}: max err {mx:.3e} mean {mean:.3e}, largest excess over the bound {worst:.3e} (tol {tol})"
    return mx, mean
