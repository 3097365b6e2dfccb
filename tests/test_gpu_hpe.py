"""GPU parity of hdt_hpe against the fp64 oracle (fp32 <= 1e-4, bf16 within bf16 rounding)."""
import numpy as np
import pytest
import torch

import gen
from gpu_util import check_close, dev_struct
from oracle import hpe_oracle as ho

pytestmark = pytest.mark.gpu


def run(P, b, d_model, n_levels, dtype, max_stages=8):
    lv, pa, cu = dev_struct(b)
    idx = P.hdt_build_index(lv, pa, cu, max_stages=max_stages)
    want = ho.hpe(b.level, b.parent, b.cu_seqlens, d_model, n_levels)
    got = P.hdt_hpe(idx, lv, pa, cu, d_model, n_levels, dtype=dtype).float().cpu().numpy().astype(np.float64)
    tol = 1e-4 if dtype == torch.float32 else 2e-2
    assert np.abs(got - want).max() <= tol
    # accumulate: x + HPE
    x0 = torch.randn((b.total_tokens, d_model), device="cuda").to(dtype)
    x = x0.clone()
    P.hdt_hpe(idx, lv, pa, cu, d_model, n_levels, x=x, accumulate=True)
    pad = torch.from_numpy(b.level < 0).cuda()
    assert torch.equal(x[pad], x0[pad])
    # bf16: x0 + HPE reaches 4 and more, where the bf16 grid is coarser than 2e-2: half an ulp of the
    # expected sum (the rounding of the stored result) is allowed on top, element by element
    check_close(x.float().cpu().numpy(), x0.float().cpu().numpy().astype(np.float64) + want,
                "f32" if dtype == torch.float32 else "bf16", "x + HPE", out_rounding=True)
    P.hdt_device_status()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_hpe_small_and_generic(dtype):
    import paper_2407_08330_b200 as P
    for seed in range(3):
        run(P, gen.small_random_batch(seed, n_seqs=4, max_len=400, K=(0, 40)), 64, 3, dtype)
    rng = np.random.default_rng(4)
    b = gen.pack([gen.layout_tree(gen.random_tree(rng, int(rng.integers(2, 7)), 5)) for _ in range(10)])
    run(P, b, 96, 6, dtype)
    run(P, b, 6, 2, dtype)          # fewer levels than the trees have: deeper levels are ignored


def test_hpe_config_sizes():
    import paper_2407_08330_b200 as P
    run(P, gen.make_hierarchy(1), 768, 3, torch.float32)
    run(P, gen.make_hierarchy(5), 768, 3, torch.float32, max_stages=4)   # sibling numbers up to ~1000


def test_hpe_sibling_numbers_from_every_index_path():
    """The index build writes the sibling numbers that hdt_hpe reads: from the per-stage kernels (a
    caller that allows more than 8 stages, or more than 1024 sequences) and from the one-CTA builder
    of the upper stages with a stage in shared memory and with one too large for it."""
    import paper_2407_08330_b200 as P
    rng = np.random.default_rng(9)
    deep = gen.pack([gen.layout_tree(gen.random_tree(rng, int(rng.integers(2, 7)), 5)) for _ in range(12)])
    run(P, deep, 64, 6, torch.float32, max_stages=24)                   # per-stage kernels on every stage
    many = gen.pack([gen.gen_fill(rng, int(rng.integers(3, 40)), (1, 3), (1, 3), (0, 6))[:2] for _ in range(1100)])
    run(P, many, 32, 3, torch.float32, max_stages=4)                    # more sequences than the one-CTA builder takes
    big = gen.pack([gen.gen_fill(rng, 30000, (4, 24), (3, 20), (2, 6)) for _ in range(2)])
    run(P, big, 32, 3, torch.float32, max_stages=4)                     # stage 1 of about 10 000 elements: global scratch
