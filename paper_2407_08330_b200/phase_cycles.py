"""Diagnostic: cycles per phase of the persistent stage-0 kernels, from their own clock stamps.

    python -m paper_2407_08330_b200.phase_cycles [config]

Thread 0 of CTA 0 of `k_fwd_tc_p` (forward, option no_persistent = 2) and of `k_bwd_tc_p`
(backward, the default at head_dim 64) accumulates clock64() differences between fixed points of
its item loop; `hdt_debug_fwd_phase_cycles` / `hdt_debug_bwd_phase_cycles` read and reset the
counters.  The numbers are one thread's view of a lockstep loop: a phase that ends in a CTA
barrier includes the wait for the slowest warp.
"""
import ctypes as C
import sys

import numpy as np
import torch

import gen
import paper_2407_08330_b200 as P

BWD_PHASES = ["loop top (row statistics of the next item)", "wait for S, dP (+ staged tiles gone)", "P, dS arithmetic",
              "barrier", "issue S, dP of the next item", "wait for the output MMAs", "input request + drain of dQ, dK, dV",
              "barrier", "TMA store requests", "item bookkeeping (next item)", "issue of the output MMAs",
              "wait for the next item's inputs"]


def main(c=3):
    cfg, b = gen.CONFIGS[c], gen.make_hierarchy(c)
    T, H, d = b.total_tokens, cfg.heads, cfg.head_dim
    t = gen.make_tensors(1, T, H, d, "bf16")
    torch.cuda.set_stream(torch.cuda.Stream())
    dev = lambda x: torch.from_numpy(x).cuda().to(torch.bfloat16)
    idx = P.hdt_build_index(torch.from_numpy(b.level).cuda(), torch.from_numpy(b.parent).cuda(),
                            torch.from_numpy(b.cu_seqlens).cuda())
    q, k, v, do = (dev(t[n]) for n in ("q", "k", "v", "do"))
    o, lse = P.hdt_attn_fwd(idx, q, k, v)
    L = P.lib()
    out = (C.c_int64 * 16)()
    for _ in range(3):
        P.hdt_attn_bwd(idx, q, k, v, o, lse, do)
    L.hdt_debug_bwd_phase_cycles(out)           # reset after the warm-up calls
    for _ in range(5):
        P.hdt_attn_bwd(idx, q, k, v, o, lse, do)
    torch.cuda.synchronize()
    L.hdt_debug_bwd_phase_cycles(out)
    v_ = np.array(list(out), float)
    n = max(v_[12], 1.0)
    print(f"backward, {cfg.name}: {int(n)} items of CTA 0, {v_[:12].sum() / n:.0f} cycles per item")
    for name, x in zip(BWD_PHASES, v_[:12] / n):
        print(f"  {name:44s} {x:7.0f}")


if __name__ == "__main__":
    main(int(sys.argv[1]) if len(sys.argv) > 1 else 3)
