#!/usr/bin/env python
"""Benchmark of the HDT hierarchical-attention hot path on B200.

One step = hdt_build_index + hdt_attn_fwd + hdt_attn_bwd over one batch of synthetic
hierarchical documents.  The headline workload is the largest forward + backward configuration and
the only one above the ridge of the measured roofline (config 5: 2 documents of 32768 tokens with
families of up to 1025 tokens, 12 heads x 64, bf16); the same JSON line carries the full record of
configs 3, 4 and 2 under "configs" (config 3 is the shape of the paper's single-layer efficiency
protocol: batch 4, 12 heads x 64).  Prints ONE JSON line on rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]
                  [--also 3,4,2] [--no-sustained] [--no-e2e] [--no-cpu-baseline] [--no-next-rows]

N > 1 (under torch.distributed.run): every rank runs an independent replica of the batch; there
is no collective on the data path (the path does not shard inside a sequence).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import gen  # noqa: E402

METRIC = "HDT attention fwd+bwd effective TFLOP/s (unmasked pairs) and % of bf16 peak; tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM traffic (read + write bytes per launch) of the kernels from ncu captures: written next to the
# profile summaries by whoever takes a capture, one entry per (workload, kernel scope) with the
# kernel's name and the commit it was built from; a scope without an entry reports null.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "traffic.json")


def ncu_traffic(workload, scope):
    try:
        for e in json.load(open(TRAFFIC_FILE))["entries"]:
            if e["workload"] == workload and e["scope"] == scope:
                return {"bytes": e["dram_bytes"], "kernel": e["kernel"], "commit": e["commit"]}
    except Exception:
        pass
    return None


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def workload(c):
    cfg = gen.CONFIGS[c]
    b = gen.make_hierarchy(c)
    return cfg, b


def max_over_ranks(x, dev):
    """Largest value of x over the ranks of the default process group (x itself without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(flops_per_replica, world, ms):
    """Whole-job effective TFLOP/s of `world` independent replicas that all finish within `ms`."""
    return flops_per_replica * world / (ms * 1e-3) / 1e12


def flops_per_step(nnz, H, d, backward):
    return (4 + (10 if backward else 0)) * d * nnz * H


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, torch_dev):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self._nv = pynvml
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(torch_dev).uuid)
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                vis = os.environ.get("CUDA_VISIBLE_DEVICES")
                idx = int(vis.split(",")[torch_dev]) if vis and vis.split(",")[0].isdigit() else torch_dev
                self._h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None
        self._t = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)) if hasattr(
                    nv, "nvmlDeviceGetCurrentClocksEventReasons") else int(
                    nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for bit, name in self.REASONS.items():
                    if bits & bit and name != "gpu_idle":
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.002)

    def __enter__(self):
        if self._h is not None:
            self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._h is not None:
            self._t.join(timeout=2)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": int(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------
def oracle_sample(c, cfg, b, heads=None, seqs=None):
    """Sub-batch of the workload for the oracle: the listed sequences and the first `heads` heads."""
    seqs = list(range(b.batch)) if seqs is None else seqs
    parts = [(b.level[b.cu_seqlens[s]:b.cu_seqlens[s + 1]], b.parent[b.cu_seqlens[s]:b.cu_seqlens[s + 1]])
             for s in seqs]
    sub = gen.pack(parts)
    H = cfg.heads if heads is None else heads
    t = gen.make_tensors(cfg.tensor_seed, sub.total_tokens, H, cfg.head_dim, cfg.dtype)
    return sub, t, H


def oracle_step(sub, t, backward, directions=7):
    import oracle
    t0 = time.perf_counter()
    oracle.forward(sub.level, sub.parent, sub.cu_seqlens, t["q"], t["k"], t["v"], directions=directions)
    if backward:
        oracle.backward(sub.level, sub.parent, sub.cu_seqlens, t["q"], t["k"], t["v"], t["do"], directions=directions)
    return time.perf_counter() - t0


def oracle_nnz(sub, directions=7):
    """Unmasked pairs of the batch from counts alone: the diagonal, one entry per non-root token
    for each of the child->parent and parent->child groups, c (c - 1) sibling entries per family
    of c children."""
    nnz = 0
    for s in range(sub.batch):
        lo, hi = sub.cu_seqlens[s], sub.cu_seqlens[s + 1]
        pa = sub.parent[lo:hi]
        real = sub.level[lo:hi] >= 0
        c = np.bincount(pa[(pa >= 0) & real], minlength=hi - lo).astype(np.int64)
        non_root = int(((pa >= 0) & real).sum())
        nnz += int(real.sum()) + non_root * (bool(directions & 1) + bool(directions & 4))
        if directions & 2:
            nnz += int((c * (c - 1)).sum())
    return nnz


CPU_SAMPLES = {2: dict(seqs=None, heads=None), 3: dict(seqs=None, heads=None),
               4: dict(seqs=[0, 1], heads=4), 5: dict(seqs=[0], heads=2), 1: dict(seqs=None, heads=None),
               6: dict(seqs=None, heads=None), 7: dict(seqs=None, heads=None)}


def cpu_baseline(c, cfg, b, directions=7):
    import oracle
    spec = CPU_SAMPLES[c]
    sub, t, H = oracle_sample(c, cfg, b, spec["heads"], spec["seqs"])
    dt = oracle_step(sub, t, cfg.backward, directions)
    fl = flops_per_step(oracle_nnz(sub, directions), H, cfg.head_dim, cfg.backward)
    return {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": oracle.threads(), "kind": "oracle",
            "sample": f"{sub.batch} of {b.batch} sequences ({sub.total_tokens} tokens), {H} of {cfg.heads} heads, "
                      f"forward{'+backward' if cfg.backward else ''} once, {dt:.2f} s",
            "tokens_per_s": sub.real_tokens / dt * (H / cfg.heads)}


def prefix_sample(c, cfg, b, n_tokens, heads):
    """The first n_tokens tokens of sequence 0 (a prefix of a document in document order is a valid hierarchy:
    parents precede their children) with the first `heads` heads of the workload's tensors."""
    lo = int(b.cu_seqlens[0])
    n = min(int(n_tokens), int(b.cu_seqlens[1]) - lo)
    sub = gen.pack([(b.level[lo:lo + n], b.parent[lo:lo + n])])
    t = gen.make_tensors(cfg.tensor_seed, sub.total_tokens, heads, cfg.head_dim, cfg.dtype)
    return sub, t


def run_reference(args):
    """The oracle as the reference arm: each step is a bounded sample of the workload — sequence 0, or a prefix
    of it, with as many heads as keep the whole run of steps + warmup within about two minutes."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    c = args.config
    cfg, b = workload(c)
    total = args.steps + args.warmup
    budget = 120.0 / max(total, 1)          # seconds per step
    dirs = args.directions
    n0 = int(b.cu_seqlens[1] - b.cu_seqlens[0])
    # grow the prefix (one head) while a step fits the budget; then add heads
    n, t1 = min(n0, 256), None
    while True:
        sub, t = prefix_sample(c, cfg, b, n, 1)
        t1 = oracle_step(sub, t, cfg.backward, dirs)
        if n >= n0 or t1 * 4.0 > budget:        # (doubling the prefix costs up to four times as much: the mask is n x n)
            break
        n = min(n0, 2 * n)
    heads = int(max(1, min(cfg.heads, budget // max(t1, 1e-4))))
    sub, t = prefix_sample(c, cfg, b, n, heads)
    H = heads
    for _ in range(args.warmup):
        oracle_step(sub, t, cfg.backward, dirs)
    times = [oracle_step(sub, t, cfg.backward, dirs) for _ in range(args.steps)]
    dt = float(np.mean(times))
    fl = flops_per_step(oracle_nnz(sub, dirs), H, cfg.head_dim, cfg.backward)
    val = fl / dt / 1e12
    sample = (f"first {sub.total_tokens} of the {n0} tokens of sequence 0 (of {b.batch} sequences), {H} of {cfg.heads} heads, "
              f"forward{'+backward' if cfg.backward else ''} per step")
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "description": cfg.description, "heads": cfg.heads,
                       "head_dim": cfg.head_dim, "sample": sample},
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": oracle.threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "tokens_per_s": sub.real_tokens / dt * (H / cfg.heads), "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
def pctl(x, q):
    return float(np.percentile(np.asarray(x, np.float64), q))


class Workload:
    """One configuration resident on the device: structure arrays, tensors, outputs, workspaces."""

    def __init__(self, P, c, args, dev, rank):
        import torch
        self.P, self.c, self.args, self.dev = P, c, args, dev
        self.cfg, self.b = workload(c)
        cfg, b = self.cfg, self.b
        self.T, self.H, self.d = b.total_tokens, cfg.heads, cfg.head_dim
        T, H, d = self.T, self.H, self.d
        self.tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
        t = gen.make_tensors(cfg.tensor_seed + rank, T, H, d, cfg.dtype)

        def pin(x, dt=None):
            h = torch.from_numpy(np.ascontiguousarray(x))
            if dt is not None:
                h = h.to(dt)
            return h.pin_memory()

        self.h_level, self.h_parent, self.h_cu = pin(b.level), pin(b.parent), pin(b.cu_seqlens)
        self.h_q, self.h_k, self.h_v, self.h_do = (pin(t[n], self.tdt) for n in ("q", "k", "v", "do"))
        del t
        self.level, self.parent, self.cu = self.h_level.to(dev), self.h_parent.to(dev), self.h_cu.to(dev)
        self.q, self.k, self.v, self.do = self.h_q.to(dev), self.h_k.to(dev), self.h_v.to(dev), self.h_do.to(dev)
        self.o = torch.empty_like(self.q)
        self.lse = torch.empty((H, T), dtype=torch.float32, device=dev)
        self.dq, self.dk, self.dv = (torch.empty_like(self.q) for _ in range(3))
        self.max_st = 24 if c == 7 else 4      # expression trees reach depth 20
        self.ws_index = torch.empty(P.hdt_index_workspace_bytes(b.batch, T, 0, self.max_st), dtype=torch.uint8, device=dev)
        idx0 = P.hdt_build_index(self.level, self.parent, self.cu, max_stages=self.max_st, workspace=self.ws_index,
                                 directions=args.directions)
        self.nnz, self.visited, self.n_stages = idx0.nnz, idx0.visited, idx0.n_stages
        self.ws_f = torch.empty(max(256, P.hdt_attn_workspace_bytes(idx0, H, d, self.tdt, 0)), dtype=torch.uint8, device=dev)
        self.ws_b = torch.empty(max(256, P.hdt_attn_workspace_bytes(idx0, H, d, self.tdt, 1)), dtype=torch.uint8, device=dev)
        del idx0
        self.flops = flops_per_step(self.nnz, H, d, cfg.backward)

    def step(self, S=None):
        P, a = self.P, self.args
        S = self.__dict__ if S is None else S
        idx = P.hdt_build_index(S["level"], S["parent"], S["cu"], max_stages=self.max_st, workspace=self.ws_index,
                                directions=a.directions, deferred=not a.waiting_build)
        P.hdt_attn_fwd(idx, S["q"], S["k"], S["v"], out=S["o"], lse=S["lse"], workspace=self.ws_f)
        if self.cfg.backward:
            P.hdt_attn_bwd(idx, S["q"], S["k"], S["v"], S["o"], S["lse"], S["do"], dq=S["dq"], dk=S["dk"], dv=S["dv"],
                           workspace=self.ws_b)
        idx.close()


def timed(fn, steps, flush):
    """Per-step CUDA events on the launch stream; with `flush` a 256 MiB write (untimed) empties L2 before every step."""
    import torch
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, z in ev:
        if flush is not None:
            flush.zero_()
        a.record()
        fn()
        z.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(z) for a, z in ev]


def kernel_times(P, W, steps, flush):
    """Device time per kernel scope from the library's own CUDA events, in a pass of `steps` steps after the timed region."""
    import ctypes as C
    L = P.lib()
    L.hdt_profile_enable(1)
    for i in range(6):
        L.hdt_profile_read(i, None, None, 1)
    for _ in range(2):
        flush.zero_()
        W.step()
    for i in range(6):
        L.hdt_profile_read(i, None, None, 1)
    timed(W.step, steps, flush)
    kern = {}
    L.hdt_profile_name.restype = C.c_char_p
    for i in range(6):
        n_, ms_ = C.c_int64(), C.c_double()
        L.hdt_profile_read(i, C.byref(n_), C.byref(ms_), 1)
        if n_.value:
            kern[L.hdt_profile_name(i).decode()] = {"launches_per_step": n_.value / steps, "ms_per_step": ms_.value / steps}
    L.hdt_profile_enable(0)
    return kern


def roofline_of(W, kern, pk):
    """Roofline of the scope that takes the most device time: achieved algorithmic bytes (or FLOP) per second
    against the measured peak that binds it."""
    cfg, real, H, d = W.cfg, W.b.real_tokens, W.H, W.d
    esz = 2 if cfg.dtype == "bf16" else 4
    # backward stage 0: q, k, v, dO in, dq, dk, dv out, lse and delta; without a delta pass (the kernel computes
    # dO . O itself) it reads o instead of delta
    fused_delta = cfg.backward and "k_delta" not in kern
    alg_bytes = {"k_fwd_stage0": (4 * d * esz + 4) * real * H,
                 "k_bwd_stage0": ((8 * d * esz + 4) if fused_delta else (7 * d * esz + 8)) * real * H,
                 "k_delta": (2 * d * esz + 4) * real * H}
    for kk in kern:
        if kk in alg_bytes:
            kd = kern[kk]["ms_per_step"] * 1e-3
            kern[kk]["achieved_gbs"] = alg_bytes[kk] / kd / 1e9
            kern[kk]["frac_of_hbm_peak"] = kern[kk]["achieved_gbs"] / pk["hbm_gbs"]
    dom = max((kk for kk in kern if kk in alg_bytes), key=lambda kk: kern[kk]["ms_per_step"], default=None)
    if dom is None:
        return None
    dur = kern[dom]["ms_per_step"] * 1e-3      # all launches of the scope in a step
    tr = ncu_traffic(cfg.name, dom)
    ach = alg_bytes[dom] / dur / 1e9
    roof = {"kernel": dom, "bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"],
            "traffic": tr["bytes"] if tr else None, "traffic_source": tr, "peak_source": pk["_source"],
            "algorithmic_bytes_per_launch": alg_bytes[dom], "kernel_ms": dur * 1e3}
    # a scope whose algorithmic intensity lies above the ridge of the two measured peaks is bound by the tensor
    # pipe (config 5: long families), not by HBM: report it against the bf16 peak (sustained figure: the kernel is
    # timed inside a step), in effective FLOP (unmasked pairs of all stages; the stages above 0 hold about 3 % of them)
    alg_flops = {"k_fwd_stage0": 4 * d * W.nnz * H, "k_bwd_stage0": 10 * d * W.nnz * H}
    tf_peak = pk.get("bf16_tflops_sustained") or pk["bf16_tflops"]
    if dom in alg_flops and alg_flops[dom] / alg_bytes[dom] > tf_peak * 1e12 / (pk["hbm_gbs"] * 1e9):
        ach_tf = alg_flops[dom] / dur / 1e12
        roof.update({"bound": "tensor", "achieved": ach_tf, "peak": tf_peak, "unit": "TFLOP/s", "frac": ach_tf / tf_peak,
                     "algorithmic_flops_per_launch": alg_flops[dom]})
    return roof


def measure(P, W, args, dev, world, flush, pk, barrier, headline):
    """Cold-L2 timed region of exactly args.steps steps (the contract's number), hot-L2 figures beside it, the
    per-kernel split and the roofline."""
    import torch
    local = dev.index
    for _ in range(args.warmup):
        flush.zero_()
        W.step()
    barrier()
    l0 = P.hdt_launch_count()
    with ClockSampler(local) as clk:
        w0 = time.perf_counter()
        times = timed(W.step, args.steps, flush)
        barrier()
        wall = time.perf_counter() - w0
    launches = P.hdt_launch_count() - l0
    ms = max_over_ranks(float(np.sum(times)) / args.steps, dev)
    hot = timed(W.step, args.steps, None)          # the same steps back to back: inputs that fit stay in L2
    kern = kernel_times(P, W, min(args.steps, 20), flush)
    roof = roofline_of(W, kern, pk)
    cfg, b = W.cfg, W.b
    value = job_value(W.flops, world, ms)
    rec = {
        "value": value, "unit": "TFLOP/s", "ms_per_step": ms,
        "ms_per_step_stats": {"median": pctl(times, 50), "p10": pctl(times, 10), "p90": pctl(times, 90), "min": float(np.min(times))},
        "hot_l2": {"ms_per_step": float(np.mean(hot)), "median": pctl(hot, 50), "value": job_value(W.flops, world, float(np.mean(hot))),
                   "note": "no flush between steps: whatever of the working set fits the 126 MB L2 stays there"},
        "pct_bf16_peak": 100.0 * value / world / pk["bf16_tflops"],
        "tokens_per_s": b.real_tokens * world / (ms * 1e-3),
        "wall_ms_per_step_incl_flush": wall / args.steps * 1e3,
        "kernels": kern, "roofline": roof, "gpu_launches": int(launches), "clocks": clk.summary(),
        "config": {"workload": cfg.name, "description": cfg.description, "batch": b.batch, "total_tokens": W.T,
                   "real_tokens": b.real_tokens, "heads": W.H, "head_dim": W.d, "nnz_pairs_per_head": W.nnz,
                   "visited_pairs_per_head": W.visited, "stages": W.n_stages, "directions": args.directions,
                   "options": args.option,
                   "step": "hdt_build_index" + ("" if args.waiting_build else " (deferred)") + " + hdt_attn_fwd" +
                           (" + hdt_attn_bwd" if cfg.backward else ""),
                   "l2": "flushed between timed steps (256 MiB write, untimed)", "parallelism": f"replicas x{world}"},
    }
    return rec


def sustained(P, W, args, dev, world, flush, seconds=2.0):
    """The same step (L2 flushed before each) repeated for at least `seconds`, with the SM clock sampled throughout:
    the figure a long job sees once the part has warmed up, and time x MHz to compare boxes of the pool."""
    import torch
    local = dev.index
    probe = float(np.mean(timed(W.step, 5, flush)))
    n = int(max(50, min(20000, seconds * 1e3 / max(probe + 0.05, 1e-3))))
    with ClockSampler(local) as clk:
        w0 = time.perf_counter()
        times = timed(W.step, n, flush)
        wall = time.perf_counter() - w0
    ms = max_over_ranks(float(np.mean(times)), dev)
    c = clk.summary()
    return {"steps": n, "wall_s": wall, "ms_per_step": ms, "median": pctl(times, 50), "p10": pctl(times, 10), "p90": pctl(times, 90),
            "value": job_value(W.flops, world, ms), "clocks": c,
            "ms_x_mhz": (ms * c["sm_mhz"]) if c.get("sm_mhz") else None}


def e2e_leg(P, W, args, dev, world, barrier):
    """End to end through the public API with host buffers (pinned): H2D of all inputs, D2H of all results, every step."""
    import torch
    cfg, b, H, T, d = W.cfg, W.b, W.H, W.T, W.d
    ho, hdq, hdk, hdv = (torch.empty_like(W.h_q).pin_memory() for _ in range(4))
    hlse = torch.empty((H, T), dtype=torch.float32).pin_memory()
    # Two sets of device buffers and three streams: the copy-in of step i + 1 and the copy-out of step i - 1 run
    # beside the compute of step i (PCIe carries both directions at once).  Every step still copies all of its
    # inputs in and all of its results out inside the timed region.
    cur = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    names = ("level", "parent", "cu", "q", "k", "v", "do", "o", "lse", "dq", "dk", "dv")
    sets = [{n: getattr(W, n) for n in names}]
    sets.append({n: torch.empty_like(t_) for n, t_ in sets[0].items()})
    ev_in = [torch.cuda.Event() for _ in range(2)]       # inputs of set j have arrived
    ev_c = [torch.cuda.Event() for _ in range(2)]        # compute on set j is done
    ev_out = [torch.cuda.Event() for _ in range(2)]      # results of set j have left
    for e in ev_c + ev_out:
        e.record(cur)

    def copy_in(j):
        S = sets[j]
        s_in.wait_event(ev_c[j])                          # the step that last used set j is done with its inputs
        with torch.cuda.stream(s_in):
            S["level"].copy_(W.h_level, non_blocking=True); S["parent"].copy_(W.h_parent, non_blocking=True)
            S["cu"].copy_(W.h_cu, non_blocking=True)
            S["q"].copy_(W.h_q, non_blocking=True); S["k"].copy_(W.h_k, non_blocking=True); S["v"].copy_(W.h_v, non_blocking=True)
            if cfg.backward:
                S["do"].copy_(W.h_do, non_blocking=True)
            ev_in[j].record(s_in)

    def compute(j):
        cur.wait_event(ev_in[j])
        cur.wait_event(ev_out[j])                         # the previous results of set j have been copied out
        W.step(sets[j])
        ev_c[j].record(cur)

    def copy_out(j):
        S = sets[j]
        s_out.wait_event(ev_c[j])
        with torch.cuda.stream(s_out):
            ho.copy_(S["o"], non_blocking=True); hlse.copy_(S["lse"], non_blocking=True)
            if cfg.backward:
                hdq.copy_(S["dq"], non_blocking=True); hdk.copy_(S["dk"], non_blocking=True)
                hdv.copy_(S["dv"], non_blocking=True)
            ev_out[j].record(s_out)

    def run_e2e(n):
        copy_in(0)
        for i in range(n):
            if i + 1 < n:
                copy_in((i + 1) & 1)
            compute(i & 1)
            copy_out(i & 1)
        s_out.synchronize()

    run_e2e(3)
    barrier()
    n_e = max(4, min(args.steps, 50))    # the first copy-in and the last copy-out are not hidden
    w0 = time.perf_counter()
    run_e2e(n_e)
    barrier()
    e_ms = max_over_ranks((time.perf_counter() - w0) / n_e * 1e3, dev)
    esz = W.q.element_size()
    n_in = 3 + (1 if cfg.backward else 0)
    n_out = 1 + (3 if cfg.backward else 0)
    return {"value": job_value(W.flops, world, e_ms), "unit": "TFLOP/s",
            "h2d_bytes_per_step": n_in * T * H * d * esz + T * 5 + (b.batch + 1) * 4,
            "d2h_bytes_per_step": n_out * T * H * d * esz + H * T * 4, "ms_per_step": e_ms, "steps": n_e,
            "pipeline": "copy-in of step i+1 and copy-out of step i-1 beside the compute of step i (two buffer sets)"}


def next_rows(P, W, args, dev, flush, pk):
    """The step before the path (hierarchical positional encoding added to a resident embedding) and the step
    after it (decoder rows cross-attending to a level subset of this batch's encoder rows), timed alone."""
    import torch
    b, H, d, T, tdt = W.b, W.H, W.d, W.T, W.tdt
    out = {}
    d_model = H * d
    x = torch.zeros((T, d_model), dtype=tdt, device=dev)
    idx = P.hdt_build_index(W.level, W.parent, W.cu, max_stages=W.max_st, workspace=W.ws_index, directions=args.directions)
    ws_h = torch.empty(max(256, P.hdt_hpe_workspace_bytes(idx, 3)), dtype=torch.uint8, device=dev)

    def step_hpe():
        P.hdt_hpe(idx, W.level, W.parent, W.cu, d_model, n_levels=3, x=x, accumulate=True, workspace=ws_h)

    n = min(args.steps, 20)
    for _ in range(3):
        step_hpe()
    l1 = P.hdt_launch_count()
    hpe_ms = float(np.mean(timed(step_hpe, n, flush)))
    hpe_bytes = 2 * T * d_model * x.element_size() + T * 5
    out["hpe"] = {"ms": hpe_ms, "algorithmic_bytes": hpe_bytes, "achieved_gbs": hpe_bytes / (hpe_ms * 1e-3) / 1e9,
                  "frac_of_hbm_peak": hpe_bytes / (hpe_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                  "launches": (P.hdt_launch_count() - l1) // n, "d_model": d_model, "levels": 3, "mode": "x += HPE(p)"}
    idx.close()
    del x, ws_h
    if W.cfg.backward:
        nq = 256
        cuq = torch.arange(0, (b.batch + 1) * nq, nq, dtype=torch.int32, device=dev)
        Tq = b.batch * nq
        gq = torch.Generator(device="cpu").manual_seed(W.cfg.tensor_seed + 77)
        xq, xdo = (torch.randn((Tq, H, d), generator=gq).to(tdt).to(dev) for _ in range(2))
        xo = torch.empty_like(xq); xlse = torch.empty((H, Tq), dtype=torch.float32, device=dev)
        xdq = torch.empty_like(xq)
        ws_x = torch.empty(max(P.hdt_cross_workspace_bytes(b.batch, T, Tq, H, d, tdt, w_) for w_ in (0, 1)),
                           dtype=torch.uint8, device=dev)
        cross = {"decoder_rows": Tq, "subsets": {}}
        for name, mask in (("[SEC]", 2), ("[SEC]+[SENT]", 6), ("[SEC]+[SENT]+tokens", 14)):
            n_keys = int(sum(int((b.level == l).sum()) for l in range(4) if (mask >> l) & 1))

            def step_x():
                P.hdt_cross_attn_fwd(W.level, W.cu, cuq, mask, xq, W.k, W.v, out=xo, lse=xlse, workspace=ws_x)
                P.hdt_cross_attn_bwd(W.level, W.cu, cuq, mask, xq, W.k, W.v, xo, xlse, xdo, dq=xdq, dk=W.dk, dv=W.dv, workspace=ws_x)

            for _ in range(2):
                step_x()
            x_ms = float(np.mean(timed(step_x, n, flush)))
            pairs = sum(nq * int(((b.level[b.cu_seqlens[s]:b.cu_seqlens[s + 1]] >= 0) &
                                  (((mask >> np.maximum(b.level[b.cu_seqlens[s]:b.cu_seqlens[s + 1]], 0)) & 1) == 1)).sum())
                        for s in range(b.batch))
            cross["subsets"][name] = {"chosen_keys": n_keys, "ms_fwd_bwd": x_ms, "tflops": 14 * d * pairs * H / (x_ms * 1e-3) / 1e12}
        out["cross_attention"] = cross
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", type=int, default=5, choices=[1, 2, 3, 4, 5, 6, 7],
                    help="the headline workload (default 5: the largest forward + backward configuration)")
    ap.add_argument("--also", default=None,
                    help="comma-separated configurations whose full record goes under \"configs\" (default 3,4,2 with --config 5, none otherwise)")
    ap.add_argument("--directions", type=int, default=7, choices=range(8),
                    help="bits 1|2|4 keep the child->parent, sibling, parent->child entries (7 = full rule)")
    ap.add_argument("--impl", default="hdt", choices=["hdt", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sustained", action="store_true")
    ap.add_argument("--no-next-rows", "--no-hpe", dest="no_next_rows", action="store_true",
                    help="skip the positional-encoding and cross-attention timings")
    ap.add_argument("--waiting-build", action="store_true",
                    help="hdt_build_index waits for the index itself (default: deferred build, the forward waits)")
    ap.add_argument("--option", action="append", default=[], metavar="NAME=VALUE",
                    help="library switch for A/B runs (hdt_set_option), e.g. bwd_walk=1")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    args.warmup = max(args.warmup, 3)

    import torch
    import torch.distributed as dist

    import paper_2407_08330_b200 as P

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    # everything runs on an explicit stream (the legacy default stream cannot be captured into the
    # CUDA graph hdt_build_index replays)
    torch.cuda.set_stream(torch.cuda.Stream(device=dev))
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for kv in args.option:
        name, _, val = kv.partition("=")
        P.hdt_set_option(name, int(val))
    pk = peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # > 126 MB L2
    c = args.config
    also = [int(x) for x in args.also.split(",") if x] if args.also is not None else ([3, 4, 2] if c == 5 else [])
    also = [x for x in also if x != c]

    W = Workload(P, c, args, dev, rank)
    head = measure(P, W, args, dev, world, flush, pk, barrier, True)
    sus = None if args.no_sustained else sustained(P, W, args, dev, world, flush)
    e2e = None if args.no_e2e else e2e_leg(P, W, args, dev, world, barrier)
    nxt = None
    if rank == 0 and not args.no_next_rows:
        nxt = next_rows(P, W, args, dev, flush, pk)
    cpu = None
    if rank == 0 and not args.no_cpu_baseline:
        cpu = cpu_baseline(c, W.cfg, W.b, args.directions)
    del W
    torch.cuda.empty_cache()
    others = {}
    for x in also:                     # the other configurations: the same measurement, one after the other
        Wx = Workload(P, x, args, dev, rank)
        others[Wx.cfg.name] = measure(P, Wx, args, dev, world, flush, pk, barrier, False)
        del Wx
        torch.cuda.empty_cache()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    line = {"metric": METRIC, "value": head["value"], "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": gen.CONFIGS[c].dtype, "data": "synthetic"}
    for k_ in ("config", "ms_per_step_stats", "hot_l2", "pct_bf16_peak", "tokens_per_s", "wall_ms_per_step_incl_flush",
               "kernels", "roofline"):
        line[k_] = head[k_]
    line["sustained"] = sus
    line["e2e"] = e2e
    line["gpu_launches"] = head["gpu_launches"]
    line["clocks"] = head["clocks"]
    if nxt:
        line["next_rows"] = nxt
    if cpu:
        line["cpu_baseline"] = cpu
    if others:
        line["configs"] = others
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
