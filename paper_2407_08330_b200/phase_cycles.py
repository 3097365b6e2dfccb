"""Diagnostic: where the looping stage-0 backward kernel spends its time, from its own clock stamps.

    python -m paper_2407_08330_b200.phase_cycles [config]
    python -m paper_2407_08330_b200.phase_cycles 5 mc      (the multi-chunk forward's chunk loop)

With option "phase_stamps" the looping forward and the transposed looping backward (head_dim 64) run
instrumented instantiations: thread 0 of CTA 0 adds clock64() differences between fixed points of
its item loop (`hdt_debug_fwd_phase_cycles` / `hdt_debug_bwd_phase_cycles` read and reset them) and every CTA records the global timer at its
entry, when its first input tiles had arrived and at the end of its loop (`hdt_debug_bwd_timeline`).
The cycle numbers are one thread's view of a lockstep loop: a phase that ends in a CTA barrier
includes the wait for the slowest warp.  With "no_persistent" = 4 the persistent 512-thread kernel
runs instead and reports its own twelve phases through the same call.
"""
import ctypes as C
import sys

import numpy as np
import torch

import gen
import paper_2407_08330_b200 as P

FWD_PHASES = ["loop top (records, ranges)", "wait for Q, K", "issue of S, wait for it", "row maximum", "exponentials, P into TMEM",
              "barrier", "wait for V, issue of P V, wait for it", "drain of O, staging", "barrier", "stores", "barrier (loop end)"]
BWD_PHASES = ["loop top (O / dO row loads, L2 prefetch of the next tiles)", "wait for the input tiles",
              "issue of S^T, dP^T", "wait for them, dO.O reduction, barrier", "P^T, dS^T arithmetic", "barrier",
              "issue of the output MMAs", "wait for dV, dK, dQ", "drain", "barrier", "TMA store requests", "loop end"]
EXTRA = {13: "  (record prefetch, inside the wait for the output MMAs)", 14: "  (row statistics prefetch, same place)"}


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
    P.hdt_set_option("phase_stamps", 1)
    try:
        L.hdt_debug_fwd_phase_cycles(out)
        for _ in range(5):
            P.hdt_attn_fwd(idx, q, k, v)
        L.hdt_debug_fwd_phase_cycles(out)
        f_ = np.array(list(out), float)
        nf = max(f_[12], 1.0)
        print(f"forward, {cfg.name}: {int(nf)} items of CTA 0, {f_[:11].sum() / nf:.0f} cycles per item")
        for name, x in zip(FWD_PHASES, f_[:11] / nf):
            print(f"  {name:60s} {x:7.0f}")
        for _ in range(3):
            P.hdt_attn_bwd(idx, q, k, v, o, lse, do)
        L.hdt_debug_bwd_phase_cycles(out)           # reset after the warm-up calls
        for i in range(16):
            out[i] = 0
        for _ in range(5):
            P.hdt_attn_bwd(idx, q, k, v, o, lse, do)
        torch.cuda.synchronize()
        L.hdt_debug_bwd_phase_cycles(out)
        v_ = np.array(list(out), float)
        n = max(v_[12], 1.0)
        print(f"backward, {cfg.name}: {int(n)} items of CTA 0, {(v_[:12].sum() + v_[13] + v_[14]) / n:.0f} cycles per item")
        for name, x in zip(BWD_PHASES, v_[:12] / n):
            print(f"  {name:60s} {x:7.0f}")
        for i, name in EXTRA.items():
            print(f"  {name:60s} {v_[i] / n:7.0f}")
        tl = (C.c_int64 * 2048)()
        L.hdt_debug_bwd_timeline(tl)
        a = np.array(list(tl), dtype=np.int64).reshape(512, 4)
        a = a[a[:, 2] > 0]
        if len(a):
            t0 = a[:, 0].min()
            st, first, end = (a[:, 0] - t0) / 1e3, (a[:, 1] - t0) / 1e3, (a[:, 2] - t0) / 1e3
            print(f"last launch, {len(a)} CTAs on {len(set(a[:, 3].tolist()))} SMs (us after the first CTA's entry): "
                  f"entry median {np.median(st):.1f} max {st.max():.1f}; first tiles in median {np.median(first):.1f}; "
                  f"end min {end.min():.1f} median {np.median(end):.1f} max {end.max():.1f}")
    finally:
        P.hdt_set_option("phase_stamps", 0)


MC_PHASES = ["wait for S (the first chunk's includes the first tiles' load)", "S into registers", "row maximum, exchange, barrier",
             "reference maximum, wait for P V of the previous chunk", "rescale of O", "exponentials, P into TMEM",
             "barrier", "issuing lane: wait for K", "issuing lane: issue of S", "issuing lane: wait for V",
             "issuing lane: issue of P V", "loop top"]


def main_mc(c=5):
    """Option "phase_stamps" = 2: thread 64 (and the issuing lane) of the eight longest blocks of head
    0 of the multi-chunk forward kernel add the cycles between fixed points of their chunk loop."""
    cfg, b = gen.CONFIGS[c], gen.make_hierarchy(c)
    T, H, d = b.total_tokens, cfg.heads, cfg.head_dim
    t = gen.make_tensors(1, T, H, d, "bf16")
    torch.cuda.set_stream(torch.cuda.Stream())
    dev = lambda x: torch.from_numpy(x).cuda().to(torch.bfloat16)
    idx = P.hdt_build_index(torch.from_numpy(b.level).cuda(), torch.from_numpy(b.parent).cuda(),
                            torch.from_numpy(b.cu_seqlens).cuda())
    q, k, v = (dev(t[n]) for n in ("q", "k", "v"))
    P.hdt_attn_fwd(idx, q, k, v)
    L = P.lib()
    out = (C.c_int64 * 16)()
    P.hdt_set_option("phase_stamps", 2)
    try:
        L.hdt_debug_fwd_phase_cycles(out)
        for _ in range(5):
            P.hdt_attn_fwd(idx, q, k, v)
        torch.cuda.synchronize()
        L.hdt_debug_fwd_phase_cycles(out)
        f_ = np.array(list(out), float)
        n = max(f_[12], 1.0)
        print(f"multi-chunk forward, {cfg.name}: {int(n)} chunks, {(f_[:7].sum() + f_[11]) / n:.0f} cycles per chunk")
        for name, x in zip(MC_PHASES, f_[:12] / n):
            print(f"  {name:62s} {x:7.0f}")
    finally:
        P.hdt_set_option("phase_stamps", 0)


if __name__ == "__main__":
    c_ = int(sys.argv[1]) if len(sys.argv) > 1 else 3
    if len(sys.argv) > 2 and sys.argv[2] == "mc":
        main_mc(c_)
    else:
        main(c_)
