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


def check_close(got, want, dtype, what):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    fin = np.isfinite(want)
    assert np.array_equal(np.isfinite(got), fin), f"{what}: finiteness differs"
    assert np.array_equal(got[~fin], want[~fin]), f"{what}: non-finite values differ"
    err = np.abs(got[fin] - want[fin])
    mx = float(err.max()) if err.size else 0.0
    mean = float(err.mean()) if err.size else 0.0
    tol = TOL[dtype]
    assert mx <= tol["max"] and mean <= tol["mean"], f"{what}: max err {mx:.3e} mean {mean:.3e} (tol {tol})"
    return mx, mean
