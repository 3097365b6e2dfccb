/*
 * libhdt — switches, test hooks and diagnostics.  Nothing here is part of the operation the paper
 * defines (none of these calls has a counterpart there); the calls of the hot path are in hdt.h.
 */
#ifndef HDT_DEBUG_H_
#define HDT_DEBUG_H_

#include "hdt.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Library options (no counterpart in the paper).  Every option is 0 by default; an unknown name
 * returns HDT_ERR_INVALID_ARG.  They exist for A/B comparisons and for tests that must reach a kernel the
 * default routing would not choose; results agree with the oracle under every setting.
 *
 *   "force_simt"     1: bf16 stage-0 work runs on the fp32 SIMT kernels, not the tensor-core ones.
 *   "simt_upper"     1: the stages above 0 of bf16 calls run on the fp32 SIMT kernels instead of the
 *                    gathering tensor-core kernels.
 *   "no_persistent"  1: only the general tensor-core kernels; 2: the persistent forward kernel (only
 *                    in a library built with HDT_WORKBENCH defined; otherwise as 0);
 *                    3: the forward kernel with one CTA per (block, head); 4: the self-contained
 *                    blocks of a head_dim 64 backward stay on the persistent 512-thread kernel
 *                    instead of the transposed looping one; 5: the looping backward kernel (the
 *                    default at head_dim 128) at head_dim 64 too; 6: one CTA per SM for the
 *                    transposed looping backward.
 *   "no_fwd_mc"      1: the blocks of a head_dim 64 forward that are not self-contained stay on the
 *                    128-thread general kernel instead of the 256-thread multi-chunk one (and with
 *                    it the EMPTY blocks of padded batches, which otherwise have a kernel of their
 *                    own, and the stages above 0 whose blocks are all self-contained, which
 *                    otherwise run in the single-chunk layout).
 *   "bwd_walk"       how a bf16 head_dim 64 backward treats the stage-0 blocks whose key range
 *                    leaves the block.  0: one walk over each block's range by the warp-specialised
 *                    kernel (dK and dV kept in tensor memory, dQ tiles summed in an fp32 buffer of
 *                    the workspace by TMA reduce-add, then scaled and rounded by a finishing pass);
 *                    1: two walks (one for dQ, one for dK and dV), no fp32 buffer; 2: the one walk
 *                    in the lock-step form of the two-walk kernel; 86: as 0, with the clock marks
 *                    that hdt_debug_bwd_w_marks and hdt_debug_bwd_w_tiles read back.
 *   "no_multi_upper" 1: where the fp32 SIMT kernels take the stages above 0 of a hierarchy of more than three
 *                    stages (fp32 calls; bf16 with "simt_upper"), a launch per stage instead of one launch
 *                    over the blocks of all of them.
 *   "no_self_beside" 1: in a backward with the one-walk kernel, the kernel of the self-contained stage-0 blocks
 *                    runs behind it on the caller's stream instead of beside it on an internal stream.
 *   "no_fused_delta" 1: the delta pass (rowsum(dO . O)) runs even where every backward kernel of the
 *                    call could compute it itself.
 *   "no_fold"        bit 0: a merge kernel completes the elements of stage 1 in the forward instead
 *                    of the stage-1 kernel itself (the default where a family of stage 1 is longer than
 *                    a block); bit 1: the stage-1 kernel does it there too; bit 2: the backward's
 *                    stage-1 kernel does the completion (off by default).
 *   "no_overlap"     1: the stages above 0 run after stage 0 on the caller's stream instead of
 *                    beside it on an internal stream.
 *   "no_graph"       1: hdt_build_index launches its kernels one by one instead of replaying a
 *                    cached CUDA graph.
 *   "no_pdl"         1: the kernels of hdt_build_index are ordinary stream successors instead of
 *                    programmatic dependents.
 *   "phase_stamps"   (only in a library built with HDT_WORKBENCH defined; otherwise ignored)
 *                    1: the instrumented instantiations of the looping forward and the transposed
 *                    looping backward (see hdt_debug_bwd_timeline); 2: that of the multi-chunk
 *                    forward (hdt_debug_fwd_phase_cycles).
 */
int hdt_set_option(const char *name, int32_t value);

/*
 * Test hook for the tensor-core primitives (no counterpart in the paper): C[128,N] = A * B on
 * one CTA with TMA-staged, 128-byte-swizzled operands and tcgen05.mma.
 *   a  device bf16 [128, K] (a_mn = 0) or [K, 128] (a_mn = 1)
 *   b  device bf16 [N, K] (b_mn = 0, C = A B^T) or [K, N] (b_mn = 1, C = A B)
 *   c  device float [128, N];  N, K multiples of 16 in 16..128.  Waits for the result.
 */
int hdt_debug_gemm(const void *a, const void *b, float *c, int32_t N, int32_t K, int32_t a_mn, int32_t b_mn,
                   void *stream);

/*
 * Test hook for the failure path of the bounded device-side waits (no counterpart in the paper).
 * Every wait of the tensor-core kernels on a completion barrier gives up after a cycle limit, raises
 * the CTA's abort flag, records HDT_ERR_TIMEOUT with the kernel and the wait site in the device
 * status word, releases its TMEM and leaves the kernel normally.  This call runs that path on one CTA
 * of 128 threads which sets up a barrier and TMEM columns as the attention kernels do and then waits,
 * for at most limit_cycles SM clock cycles (1e3..2e9), on the barrier without anything ever having
 * been issued that could arrive on it: no copy and no MMA is in flight when the wait gives up.
 * Returns what hdt_device_status(stream) reports afterwards (HDT_ERR_TIMEOUT when the path works; the
 * word is cleared, so the next call of the library runs normally); *left_early (may be NULL) receives
 * the number of threads that stopped waiting because of the abort flag rather than their own limit.
 */
int hdt_debug_wait_timeout(int64_t limit_cycles, int32_t *left_early, void *stream);

/*
 * Diagnostics (no counterpart in the paper): SM clock cycles that CTA 0 of the persistent backward
 * kernel spent in each of its phases since the last call (out16[0..11]: prefetch issue, wait for
 * S/dP, P/dS arithmetic, barrier, rest of the MMA issue, wait for dQ/dK/dV, drain, barrier, stores,
 * loop end, issue of the output MMAs, wait for the next item's TMA), out16[12] = items processed.
 * Synchronises the device and resets the counters.
 */
int hdt_debug_bwd_phase_cycles(int64_t *out16);
/* The same for the persistent forward kernel: out16[0..11] = prefetch issue, wait for S, row maximum,
 * barriers (max exchange), P arithmetic and stores, barrier, MMA issue, wait for O, drain, loop top,
 * barrier, output stores; out16[12] = items processed. */
int hdt_debug_fwd_phase_cycles(int64_t *out16);
/* With option "phase_stamps" = 1 the looping forward (head_dim 64) runs an instrumented instantiation
 * too and hdt_debug_fwd_phase_cycles reports its phases (out16[0..10]: loop top, wait for Q/K, S,
 * row maximum, exponentials with P into TMEM, barrier, V and the P V MMA, drain, barrier, stores, loop
 * end).  With the same option the transposed looping backward (head_dim 64) runs an instrumented
 * instantiation: hdt_debug_bwd_phase_cycles then reports its phases (out16[0..11]: loop top, wait for
 * the input tiles, issue of S^T/dP^T, wait for them, P^T/dS^T arithmetic, barrier, issue of the output
 * MMAs, prefetch and wait for dV/dK/dQ, drain, barrier, store requests, loop end), and
 * hdt_debug_bwd_timeline the last such launch per CTA (up to 512): out2048[4 c + 0..3] = global timer
 * (ns) at entry, when the first input tiles had arrived, at the end of the item loop, and the SM. */
int hdt_debug_bwd_timeline(int64_t *out2048);
/* The same for the last instrumented launch of the looping forward, up to 1024 CTAs. */
int hdt_debug_fwd_timeline(int64_t *out4096);

/* With option "bwd_walk" = 86: the SM clock at fixed points of tiles 20 and 21 of CTA 0 of the last launch of the
 * warp-specialised one-walk backward (families longer than a row block, head_dim 64), out128[16 role + 8 (tile - 20) + mark]; roles 0 / 1 the compute groups (marks: loop top, S^T / dP^T
 * there, other waits passed, arrived), 2 the drain group (loop top, dQ there, reduce requested), 3 the load warp
 * (before / after the wait for the ring stage), 4 the MMA warp (loop top, group a arrived, other waits passed,
 * step a issued, group b arrived, dQ accumulator free, step b issued). */
int hdt_debug_bwd_w_marks(int64_t *out128);
/* The same run: out512[t] = (SM clock << 8 | unit number mod 256) at the MMA warp's loop top of tile t of CTA 0. */
int hdt_debug_bwd_w_tiles(int64_t *out512);

/* Timing probe of the tensor pipe (allocates 16 bytes of device memory for its result and waits for the
 * device): one thread of one CTA issues `reps` groups of `per_group` MMAs (M = 128, N = n <= 128 (the probe holds two 64-column operand groups), K = 16 each; A from
 * shared memory or, a_tmem = 1, from TMEM; B K-major or, b_mn = 1, MN-major) and commits once.  out2[0] = SM
 * clock cycles from the first issue until the last MMA had completed, out2[1] = cycles of the issue loop.
 * mode bit 0: A from TMEM; bit 1: consecutive MMAs alternate between two accumulators (none depends on the one before); bit 2: two warps issue
 * the same sequence side by side (n <= 64), out2 holds the first warp's figures. */
int hdt_debug_mma_rate(int32_t n, int32_t reps, int32_t per_group, int32_t mode, int32_t b_mn, int64_t *out2);

/* Timing probe of TMEM loads (allocates 256 bytes of device memory for its result and waits for the device):
 * `warps` (1..28) warps of one CTA each run `reps` rounds of `per_round` (1..4) loads of 32 lanes x 16 columns
 * followed by one wait; with mma != 0 another warp keeps the tensor pipe busy meanwhile.  out32[w] = SM clock
 * cycles of warp w's loop. */
int hdt_debug_tmem_ld(int32_t warps, int32_t reps, int32_t per_round, int32_t mma, int64_t *out32);

#ifdef __cplusplus
}
#endif
#endif /* HDT_DEBUG_H_ */
