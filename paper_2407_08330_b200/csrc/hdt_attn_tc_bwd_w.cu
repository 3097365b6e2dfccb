// Warp-specialised one-walk backward for stage 0 in bf16 at D = 64: the row blocks that are neither
// self-contained nor EMPTY, i.e. the pieces of families longer than a row block.
//
// A unit is (row block, head).  The block is taken as KEYS only (K, V of its 128 token rows stay in
// shared memory) and walks its key span [ka, kb) — which, the family ranges being symmetric, holds
// every query that attends one of its keys — in query tiles of 128 rows, each in two steps of 64
// queries.  With the keys in the TMEM lanes (the transposed pass of hdt_attn_tc_bwd_t.cu):
//   MMA      S^T = K Q^T, dP^T = V dO^T for the step's 64 queries            -> TMEM (lane = key)
//   compute  P^T = exp2(S^T c - LSE[query]) inside the key's range, dS^T = softmax_scale P^T o (dP^T - delta[query])
//            (the factor here, in the fma that subtracts delta, so that dK and dQ need none afterwards);
//            P^T (bf16) stays in TMEM over the S^T columns it came from, dS^T -> shared memory
//   MMA      dV += P^T dO (A operand from TMEM), dK += dS^T Q: accumulated in TMEM over the whole walk;
//            after both steps dQ_tile = dS K (M = the tile's 128 queries, A = dS^T read MN-major), a
//            fresh accumulator per tile
//   drain    the dQ tile as fp32 through a swizzled staging tile and two TMA reduce-add copies into the
//            buffer a.dq_acc [T, H, 64] (k_dq_finish scales and converts the sums afterwards); at the
//            end of the unit dK, dV -> bf16 rows, staged in the unit's K / V buffer, TMA stores
// Every tile pair is visited once (the two-walk kernels compute S, dP, P, dS of each pair twice).
//
// One CTA of 736 threads per SM.  Warps 0-7 compute step a (queries 0..63 of each tile: warp = TMEM lane
// quarter x half of the step's queries), warps 8-15 step b, warps 16-19 drain, warp 20 requests the
// tiles (TMA) and fetches the queries' LSE and delta, warp 21 issues the MMAs, warp 22 requests the
// reduce-add copies of the staged dQ tiles.  The roles meet only at mbarriers, so the tensor pipe, the
// exponentials of the two compute groups, the drains and the copies overlap; S^T / dP^T are double
// buffered by step, dS^T and the dQ accumulator by tile, Q / dO by tile, K / V by unit.
// TMEM columns: S^T a 0..63 (P^T a over 0..15 and 32..47: each warp writes inside the columns it alone
// reads), dP^T a 64..127, step b the same from 128; dK 256..319, dV 320..383, dQ 384..447 and 448..511.
//
// What was measured on the way (cycles of the SM clock, one CTA per SM, config 5):
//  - one thread issuing back to back: an MMA of M = 128, K = 16 takes about 75 cycles at N = 64 with both
//    operands in shared memory (63 with two issuing warps: the pipe's own pace), 39..47 with A in TMEM,
//    106 / 70 at N = 128: the operand reads, not the arithmetic, set the pace at these shapes.  A tile
//    pair costs the tensor pipe about 2500 cycles here (32 MMAs from shared memory, 8 with A in TMEM).
//  - a round of tcgen05.ld + wait costs a warp 150 cycles alone and about 100 cycles per warp that shares
//    its TMEM lane quarter at the same time, whether the round loads 16 or 64 columns: few, wide rounds.
//  - what a compute group waits for between two of its steps is dV of the step (its P^T lies over the
//    S^T columns) and the next S^T / dP^T; dK and dQ, which read dS^T from shared memory, are issued
//    behind them.  With four warps per compute group a step's arithmetic (64 entries per thread) took
//    3500 cycles, one instruction issued in eight cycles per warp: the groups have eight warps each.
//  - the warps of an SM quarter share one instruction issue slot a cycle, and the sixteen compute warps fill most
//    of them: the MMA warp gets an instruction out every five or six cycles, so its waits, its walk and the
//    forty MMAs of a tile are a chain of 3500 cycles by themselves.  It walks tile counts only (ring stage and
//    parity from the tile number), the compute warps a record of four integers; that took the scope on config 5
//    from 0.625 to 0.589 ms together with: the drain group reads dV before dK at a unit's end and frees each with
//    a barrier of its own, so that dV and the next S^T / dP^T are issued while dK is still being read.
//    Tried and not kept: two MMA warps taking turns, the Q / dO ring in half tiles, the loop unrolled by tile
//    parity (more spills), sleeping between barrier tests in the other warps.
//  - units end often (4.7 tiles per unit on config 5): one K / V buffer cost 13000 cycles per unit
//    (the pipeline drains and refills around the reload), draining dK / dV by the compute groups with
//    plain stores 7000 (32 rows per store instruction); with the second buffer, the drain group taking
//    the accumulators first and staging them in the finished unit's K / V buffer, a unit's first tile
//    takes 4000..5000 cycles against 3500 inside a unit.
//  - the reduce-add copies of a 32 KB dQ tile take about 2500 cycles to read their staging tile; with
//    the staging in the tile's dS^T buffer every other tile waited for them (a third of the ring of
//    Q / dO tiles went to a staging area of its own instead), requested by a warp of their own because
//    the requesting thread waits for the read.  Adding the tile from registers with red.global.v4.f32
//    was much slower (the step time rose from 0.75 to 0.98 ms).
#include <cuda_bf16.h>

#include "hdt_internal.cuh"
#include "hdt_sm100.cuh"
#include "hdt_tmap.cuh"

namespace hdt {
using namespace sm100;

namespace {
constexpr int SUB = 16384;
constexpr long long WAIT_CYCLES = 400000000LL;
constexpr int KID = 7;     // kernel id in the device status word
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

// Barrier `id` over `n` threads (a warp group) that also tells every thread whether ALL of them
// passed `pred`: the group leaves its loop together when a bounded wait of one thread ran out.
__device__ __forceinline__ bool group_all(bool pred, int id, int n) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %1, 0;\n\t"
        "bar.red.and.pred q, %2, %3, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred), "r"(id), "r"(n)
        : "memory");
    return r != 0;
}

// Timeline of two tiles of CTA 0 (option "bwd_walk" = 86): absolute SM clock at fixed points of each role.
__device__ long long g_bwd_w_marks[128];
__device__ long long g_bwd_w_tiles[512];      // (instrumented run) CTA 0: SM clock at the MMA warp's loop top of every tile, unit number in the low 8 bits
#define W_MARK(role, tt, id)                                                                    \
    do {                                                                                        \
        if (MARKS && marks && (tt) >= 4 && (tt) < 6) {                                        \
            const long long now_ = clock64();                                                   \
            if (lane == 0) s_marks[(role) * 16 + ((tt) - 4) * 8 + (id)] = now_;                \
        }                                                                                       \
    } while (0)

struct WUnit { int valid, r0, r1, ka, kb, h, nt; };
// Position of a role in this CTA's sequence of query tiles: unit slot k, unit U (its uc-th non-empty
// unit), tile j of it, t-th tile overall, which lies in stage qs of the Q / dO ring on that stage's
// use of parity qph; N: the record of the unit after U, requested a unit ahead.
struct Walk { int k, j, t, uc, valid, qs, qph; WUnit U, N; };
}  // namespace

// MARKS: the instantiation that leaves the clock marks and the tile log (option "bwd_walk" = 86).
template <bool DIRS, bool MARKS = false>
__global__ void __launch_bounds__(736, 1) k_bwd_tc_w(const __grid_constant__ CUtensorMap tm_q,
                                                     const __grid_constant__ CUtensorMap tm_k,
                                                     const __grid_constant__ CUtensorMap tm_v,
                                                     const __grid_constant__ CUtensorMap tm_do,
                                                     const __grid_constant__ StoreMaps sm_out,
                                                     const __grid_constant__ CUtensorMap tm_acc, const BwdStageArgs a) {
    constexpr int D = 64;
    constexpr uint32_t TM_DK = 256, TM_DV = 320, TM_DQ = 384, TM_COLS = 512;
    constexpr int W_DRAIN = 16, W_LOAD = 20, W_MMA = 21, W_RED = 22;      // first warp of each role
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *sKV = smem_raw;                 // [2 units] x {K, V}
    uint8_t *sQD = sKV + 4 * SUB;            // [2 tiles] x {Q, dO}
    uint8_t *sDS = sQD + 4 * SUB;            // [2 tiles] x {dS^T of step a, of step b}: row = key, 64 queries per row
    uint8_t *sStg = sDS + 4 * SUB;           // staging of a dQ tile as fp32: two swizzled [128 rows x 32 columns] halves
    float2 *sStat = (float2 *)(sStg + 2 * SUB);   // [2 tiles][128]: LSE * log2(e) and delta of the tile's queries
    uint64_t *bars = (uint64_t *)(sStat + 2 * 128);
    uint64_t *qdo_full = bars, *qdo_empty = bars + 3, *sdp_full = bars + 6, *pds_ready = bars + 8;
    uint64_t *dq_full = bars + 10, *dq_free = bars + 12, *kv_full = bars + 14, *kv_empty = bars + 16;
    uint64_t *acc_full = bars + 18, *dv_free = bars + 19, *stat_full = bars + 20, *stg_free = bars + 22, *stg_full = bars + 24, *kv_reuse = bars + 26;
    uint64_t *dk_free = bars + 28, *dvacc_full = bars + 29;
    uint32_t *slot = (uint32_t *)(bars + 30);
    volatile int *abort_flag = (volatile int *)(slot + 1);
    long long *s_marks = (long long *)(bars + 31);      // [5 roles][2 tiles][8 marks] of the instrumented run (only then allocated)

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int H = a.H, G = gridDim.x;
    const float LOG2E = 1.4426950408889634f;
    const bool marks = MARKS && blockIdx.x == 0 && (warp == 0 || warp == 8 || warp == W_DRAIN || warp >= W_LOAD);
    if (MARKS && tid < 80) s_marks[tid] = 0;
    // EMPTY blocks cost nothing in the queue's order, so they are the tail of queue_split and are left
    // out here (k_dq_finish writes their rows)
    const int n_units = (a.nb - a.n_fused - a.n_empty) * H;

    if ((smem_u32(smem_raw) & 1023u) != 0u) {      // the swizzled tiles need 1024-byte alignment
        if (tid == 0) atomicCAS(a.status, 0, HDT_ERR_CUDA);
        return;
    }
    if (tid == 0) {
        for (int i = 0; i < 3; ++i) {
            mbar_init(&qdo_full[i], 1);
            mbar_init(&qdo_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sdp_full[i], 1);
            mbar_init(&pds_ready[i], 256);
            mbar_init(&dq_full[i], 1);
            mbar_init(&dq_free[i], 128);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&kv_full[i], 1);
            mbar_init(&kv_empty[i], 1);
            mbar_init(&stat_full[i], 1);
            mbar_init(&stg_free[i], 1);
            mbar_init(&stg_full[i], 128);
            mbar_init(&kv_reuse[i], 1);
        }
        mbar_init(acc_full, 1);
        mbar_init(dv_free, 128);
        mbar_init(dk_free, 128);
        mbar_init(dvacc_full, 1);
        *abort_flag = (*a.status != 0);
        fence_mbar_init();
    }
    if (warp == 0) tmem_alloc(slot, TM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *slot;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const bool dead = (*abort_flag != 0);
    bool ok = true;
    int fail_site = 0;
    // (the warp-wide instructions of every role need all lanes to take the same way: after its waits a
    // warp agrees on whether all of them ended well)
#define HDT_AGREE() (ok = __all_sync(0xffffffffu, ok))
#define HDT_WAIT(bar, parity, site)                                                   \
    do {                                                                              \
        if (ok && !mbar_wait((bar), (uint32_t)(parity), abort_flag, WAIT_CYCLES)) {   \
            ok = false;                                                               \
            fail_site = (site);                                                       \
        }                                                                             \
    } while (0)

    // ---- this CTA's sequence of units and tiles (every role walks it on its own) -------------------
    auto get_unit = [&](int k) {
        WUnit u{0, 0, 0, 0, 0, 0, 0};
        const int i = (int)blockIdx.x + k * G;
        if (i < n_units) {
            const int bi = i / H;
            const int *rec = a.blocks + 5 * (size_t)a.queue_split[a.n_fused + bi];
            u.valid = 1; u.r0 = rec[0]; u.r1 = rec[1]; u.ka = rec[2]; u.kb = rec[3]; u.h = i - bi * H;
            u.nt = (u.kb - u.ka + 127) >> 7;      // (>= 1: EMPTY blocks are not among these units)
        }
        return u;
    };
    // The record of the unit after the current one is requested a whole unit ahead (w.N): its loads
    // are in flight while the current unit is walked and no role waits for them at a unit boundary.
    auto step = [&](Walk &w) {      // to the next tile
        ++w.t;
        if (++w.qs == 2) { w.qs = 0; w.qph ^= 1; }
        if (w.uc >= 0 && w.j + 1 < w.U.nt) { ++w.j; return; }
        while (true) {
            const WUnit u = w.N;
            w.N = get_unit(w.k++);
            if (!u.valid) { w.valid = 0; return; }
            if (u.nt > 0) { w.U = u; w.j = 0; ++w.uc; w.valid = 1; return; }
        }
    };
    auto begin = [&]() {
        Walk w;
        w.k = 0; w.j = 0; w.t = -1; w.uc = -1; w.valid = 0; w.qs = 1; w.qph = 1; w.U = WUnit{0, 0, 0, 0, 0, 0, 0};
        w.N = get_unit(w.k++);
        step(w);
        return w;
    };

    if (!dead && n_units > 0) {
        if (warp == W_LOAD) {
            // ================= load warp: K / V per unit, Q / dO and the queries' statistics per tile =================
            for (Walk w = begin(); w.valid && ok; step(w)) {
                const WUnit &U = w.U;
                const int q0 = U.ka + 128 * w.j, qs = w.qs;
                // before the wait for the ring stage: the tile starts its way into L2 and the queries'
                // statistics into registers
                if (lane == 0) {
                    tma_prefetch_3d(&tm_q, 0, U.h, q0);
                    tma_prefetch_3d(&tm_do, 0, U.h, q0);
                }
                float2 st4[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = q0 + lane + 32 * i;
                    st4[i] = make_float2(0.f, 0.f);
                    if (row < U.kb) st4[i] = make_float2(a.lse[(size_t)U.h * a.T + row] * LOG2E, a.delta[(size_t)U.h * a.T + row] * a.scale);
                }
                W_MARK(3, w.t, 0);
                if (w.j == 0) {      // the unit's K, V into the buffer the unit before the last one has left
                    if (w.uc >= 2) {      // every MMA of unit uc - 2 has read the buffer, and its dK, dV rows, staged there afterwards, have left
                        HDT_WAIT(&kv_empty[w.uc & 1], ((w.uc >> 1) + 1) & 1, 1);
                        HDT_WAIT(&kv_reuse[w.uc & 1], ((w.uc >> 1) + 1) & 1, 19);
                    }
                    if (!HDT_AGREE()) break;
                    if (lane == 0) {
                        uint8_t *kv = sKV + (w.uc & 1) * 2 * SUB;
                        mbar_expect_tx(&kv_full[w.uc & 1], 2u * SUB);
                        tma_load_3d(kv, &tm_k, 0, U.h, U.r0, &kv_full[w.uc & 1]);
                        tma_load_3d(kv + SUB, &tm_v, 0, U.h, U.r0, &kv_full[w.uc & 1]);
                    }
                }
                if (w.t >= 2) HDT_WAIT(&qdo_empty[qs], w.qph ^ 1, 2);
                if (!HDT_AGREE()) break;
                W_MARK(3, w.t, 1);
                if (lane == 0) {
                    uint8_t *qd = sQD + qs * 2 * SUB;
                    mbar_expect_tx(&qdo_full[qs], 2u * SUB);
                    tma_load_3d(qd, &tm_q, 0, U.h, q0, &qdo_full[qs]);
                    tma_load_3d(qd + SUB, &tm_do, 0, U.h, q0, &qdo_full[qs]);
                }
                if (!HDT_AGREE()) break;
#pragma unroll
                for (int i = 0; i < 4; ++i) sStat[(w.t & 1) * 128 + lane + 32 * i] = st4[i];
                __syncwarp();
                if (lane == 0) mbar_arrive(&stat_full[w.t & 1]);
                if (w.j == min(1, U.nt - 1) && w.N.valid && lane == 0) {      // the next unit's K, V on their way into L2
                    tma_prefetch_3d(&tm_k, 0, w.N.h, w.N.r0);
                    tma_prefetch_3d(&tm_v, 0, w.N.h, w.N.r0);
                }
            }
        } else if (warp == W_RED) {
            // ================= reduce warp: the TMA reduce-add copies of every staged dQ tile =================
            for (Walk w = begin(); w.valid && ok; step(w)) {
                const int t = w.t;
                HDT_WAIT(&stg_full[0], t & 1, 18);
                if (!HDT_AGREE()) break;
                if (lane == 0) {
                    const uint8_t *stg = sStg;
                    const int q0 = w.U.ka + 128 * w.j;      // the tile's first query row
                    tma_reduce_add_3d(&tm_acc, 0, w.U.h, q0, stg);
                    tma_reduce_add_3d(&tm_acc, 32, w.U.h, q0, stg + SUB);
                    bulk_commit();
                    bulk_wait_read();                 // the copies have read the tile:
                    mbar_arrive(&stg_free[0]);        // the drain group may stage the next tile
                }
                __syncwarp();
            }
        } else if (warp == W_MMA) {
            // ================= MMA warp =================
            const uint32_t id_sdp = idesc_bf16(64, false, false);   // A = K / V (K-major), B = Q / dO rows of the step (K-major)
            const uint32_t id_kv = idesc_bf16(D, false, true);      // A = P^T (TMEM) / dS^T (K-major), B = dO / Q (MN-major)
            const uint32_t id_q = idesc_bf16(D, true, true);        // A = dS (MN-major: stored as dS^T), B = K (MN-major)
            // base descriptors (two 32-bit words each) of every operand form; an MMA adds (byte offset >> 4)
            // to the low word.  K-major: sbo 1024; MN-major: lbo = SUB between 64-element groups, sbo 1024.
            const uint64_t d_kv_k = smem_desc(smem_u32(sKV), 0, 1024), d_kv_mn = smem_desc(smem_u32(sKV), SUB, 1024);
            const uint64_t d_qd_k = smem_desc(smem_u32(sQD), 0, 1024), d_qd_mn = smem_desc(smem_u32(sQD), SUB, 1024);
            const uint64_t d_ds_k = smem_desc(smem_u32(sDS), 0, 1024), d_ds_mn = smem_desc(smem_u32(sDS), SUB, 1024);
            const uint32_t kvk_lo = (uint32_t)d_kv_k, kvk_hi = (uint32_t)(d_kv_k >> 32), kvm_lo = (uint32_t)d_kv_mn, kvm_hi = (uint32_t)(d_kv_mn >> 32);
            const uint32_t qdk_lo = (uint32_t)d_qd_k, qdk_hi = (uint32_t)(d_qd_k >> 32), qdm_lo = (uint32_t)d_qd_mn, qdm_hi = (uint32_t)(d_qd_mn >> 32);
            const uint32_t dsk_lo = (uint32_t)d_ds_k, dsk_hi = (uint32_t)(d_ds_k >> 32), dsm_lo = (uint32_t)d_ds_mn, dsm_hi = (uint32_t)(d_ds_mn >> 32);
            constexpr uint32_t S16 = SUB >> 4;      // one sub-tile in descriptor address units
            auto issue_sdp = [&](int x, int qs, int kvb) {
                const uint32_t q_lo = qdk_lo + qs * 2 * S16 + x * (8192 >> 4), k_lo = kvk_lo + kvb * 2 * S16;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ss_w(tmem + 128u * x, k_lo + 2 * kk, kvk_hi, q_lo + 2 * kk, qdk_hi, id_sdp, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ss_w(tmem + 128u * x + 64u, k_lo + S16 + 2 * kk, kvk_hi, q_lo + S16 + 2 * kk, qdk_hi, id_sdp, kk > 0);
                mma_commit(&sdp_full[x]);
            };
            auto issue_dv = [&](int x, int qs, uint32_t acc) {      // P^T: queries 0..31 of the step in columns 0..15, 32..63 in 32..47
                const uint32_t do_lo = qdm_lo + qs * 2 * S16 + x * (8192 >> 4) + S16;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ts_w(tmem + TM_DV, tmem + 128u * x + (kk < 2 ? 8u * kk : 32u + 8u * (kk - 2)), do_lo + 128 * kk, qdm_hi, id_kv, acc | (kk > 0));
            };
            auto issue_dk = [&](int x, int qs, int dsb, uint32_t acc) {
                const uint32_t q_lo = qdm_lo + qs * 2 * S16 + x * (8192 >> 4);
                const uint32_t d_lo = dsk_lo + dsb * 2 * S16 + x * S16;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ss_w(tmem + TM_DK, d_lo + 2 * kk, dsk_hi, q_lo + 128 * kk, qdm_hi, id_kv, acc | (kk > 0));
            };
            // (dS^T also lies packed over the dP^T columns, like P^T over S^T: dK takes it from there, which spares
            // the shared-memory pipe the 4 KB operand of each of these MMAs and is the faster form besides)
            auto issue_dk_t = [&](int x, int qs, uint32_t acc) {
                const uint32_t q_lo = qdm_lo + qs * 2 * S16 + x * (8192 >> 4);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_ts_w(tmem + TM_DK, tmem + 128u * x + 64u + (kk < 2 ? 8u * kk : 32u + 8u * (kk - 2)), q_lo + 128 * kk, qdm_hi, id_kv, acc | (kk > 0));
            };
            auto issue_dq = [&](int dsb, int kvb) {
                const uint32_t d_lo = dsm_lo + dsb * 2 * S16, k_lo = kvm_lo + kvb * 2 * S16;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ss_w(tmem + TM_DQ + 64u * dsb, d_lo + 128 * kk, dsm_hi, k_lo + 128 * kk, kvm_hi, id_q, kk > 0);
            };
            // (a walk of its own with the little this warp needs: tiles per unit, requested a unit ahead; the ring
            // stage and its parity follow from the tile count.  Every instruction here is on the kernel's
            // critical chain: the warp shares its scheduler with five others.)
            auto unit_nt = [&](int k) {
                const int i = (int)blockIdx.x + k * G;
                if (i >= n_units) return 0;
                const int *rec = a.blocks + 5 * (size_t)a.queue_split[a.n_fused + i / H];
                return (rec[3] - rec[2] + 127) >> 7;      // (>= 1: EMPTY blocks are not among these units)
            };
            int nt = unit_nt(0), nt_n = unit_nt(1), k = 2, j = 0, t = 0, uc = 0;
            if (nt > 0) {      // S^T, dP^T of both steps of the first tile
                HDT_WAIT(&kv_full[0], 0, 3);
                HDT_WAIT(&qdo_full[0], 0, 4);
                if (HDT_AGREE() && elect_one()) {
                    tc_fence_after();
                    issue_sdp(0, 0, 0);
                    issue_sdp(1, 0, 0);
                }
                __syncwarp();
            }
            while (nt > 0 && ok) {
                // the next tile: same unit or the next one (units here are never EMPTY)
                const int db = t & 1, qs = t & 1, n_qs = qs ^ 1;
                const bool first = j == 0, last = j == nt - 1;
                const bool n_valid = !last || nt_n > 0;
                const int n_qph = ((t + 1) >> 1) & 1, n_uc = uc + (last ? 1 : 0);
                const int kvb = uc & 1;
                const uint32_t acc = first ? 0u : 1u;
                // ---- step a: dV; S^T, dP^T of the next tile's step a; dK ----
                W_MARK(4, t, 0);
                if (MARKS && blockIdx.x == 0 && lane == 0 && t < 512) g_bwd_w_tiles[t] = (clock64() << 8) | (long long)(uc & 255);
                // dV of the step first: it needs nothing of the next tile.  S^T / dP^T of the next tile's step a behind
                // it (P^T lies over the S^T columns), once that tile's Q / dO are there, then dK: the pipe has dV to
                // work on while this warp waits for the load.
                if (first && uc >= 1) HDT_WAIT(dv_free, (uc - 1) & 1, 6);      // the previous unit's dV has been read (dK: below)
                W_MARK(4, t, 1);
                HDT_WAIT(&pds_ready[0], t & 1, 5);
                if (!HDT_AGREE()) break;
                W_MARK(4, t, 2);
                if (elect_one()) {
                    tc_fence_after();
                    issue_dv(0, qs, acc);
                    if (!(first && uc >= 1)) issue_dk_t(0, qs, acc);      // (before the next dP^T overwrites its operand)
                }
                __syncwarp();
                if (n_valid) {
                    HDT_WAIT(&qdo_full[n_qs], n_qph, 7);
                    if (last) HDT_WAIT(&kv_full[n_uc & 1], (n_uc >> 1) & 1, 8);      // the next tile opens a unit (the other K / V buffer)
                    if (!HDT_AGREE()) break;
                }
                if (elect_one()) {
                    tc_fence_after();
                    if (n_valid) issue_sdp(0, n_qs, n_uc & 1);
                }
                __syncwarp();
                if (first && uc >= 1) {
                    // (the drain group reads dV first: dV and the next S^T / dP^T, which the compute group waits for, have
                    // gone ahead while it still reads the previous unit's dK; this dK takes dS^T from shared memory, the
                    // copy in TMEM is gone by now)
                    HDT_WAIT(dk_free, (uc - 1) & 1, 24);
                    if (!HDT_AGREE()) break;
                    if (elect_one()) issue_dk(0, qs, db, acc);
                    __syncwarp();
                }
                W_MARK(4, t, 3);
                // ---- step b: dV; S^T, dP^T of the next tile's step b; dK; the tile's dQ ----
                if (t >= 2) HDT_WAIT(&dq_free[db], ((t >> 1) + 1) & 1, 10);
                W_MARK(4, t, 4);
                HDT_WAIT(&pds_ready[1], t & 1, 9);
                if (!HDT_AGREE()) break;
                W_MARK(4, t, 5);
                if (elect_one()) {
                    tc_fence_after();
                    issue_dv(1, qs, 1u);
                    if (last) mma_commit(dvacc_full);        // dV of the unit is complete: the drain group may start on it
                    issue_dk_t(1, qs, 1u);
                    if (n_valid) issue_sdp(1, n_qs, n_uc & 1);
                    mma_commit(&qdo_empty[qs]);        // every MMA that reads this tile's Q / dO has been issued
                    if (last) mma_commit(acc_full);
                    issue_dq(db, kvb);
                    mma_commit(&dq_full[db]);
                    if (last) mma_commit(&kv_empty[kvb]);
                }
                __syncwarp();
                W_MARK(4, t, 6);
                ++t;
                if (!last) ++j;
                else { nt = nt_n; nt_n = unit_nt(k++); j = 0; ++uc; }
            }
        } else if (warp < W_DRAIN) {
            // ================= compute groups: x = 0 (warps 0-7) step a, x = 1 (warps 8-15) step b;
            // a warp: TMEM lane quarter warp % 4, queries 32 qh .. 32 qh + 31 of the step =================
            const int x = warp >> 3, qh = (warp >> 2) & 1, kl = (warp & 3) * 32 + lane;
            const uint32_t tm_s = tmem + 128u * x + 32u * qh + lane_base, tm_dp = tm_s + 64u;
            // (a walk of its own with what a compute warp needs: the unit's rows and span, this lane's key range;
            // the next unit's are requested a unit ahead, at the unit's second tile)
            struct CU { int r0, r1, ka, kb; };
            auto unit_rec = [&](int k) {
                CU u{0, 0, 0, 0};      // (kb == ka: no such unit)
                const int i = (int)blockIdx.x + k * G;
                if (i < n_units) {
                    const int *rec = a.blocks + 5 * (size_t)a.queue_split[a.n_fused + i / H];
                    u.r0 = rec[0]; u.r1 = rec[1]; u.ka = rec[2]; u.kb = rec[3];
                }
                return u;
            };
            auto range_of = [&](const CU &u, int &lo_, int &hi_) {
                const int r = u.r0 + kl;
                lo_ = 0; hi_ = 0;
                if (u.kb > u.ka && r < u.r1) { lo_ = a.rng[2 * r]; hi_ = a.rng[2 * r + 1]; }
            };
            CU U = unit_rec(0), N = unit_rec(1);
            int k = 2, j = 0, t = 0, lo, hi, lo_n = 0, hi_n = 0;
            range_of(U, lo, hi);
            while (U.kb > U.ka && ok) {
                const int nt = (U.kb - U.ka + 127) >> 7;
                const int row = U.r0 + kl;
                const bool inb = row < U.r1;
                if (j == min(1, nt - 1)) range_of(N, lo_n, hi_n);
                const int db = t & 1;
                const int q0 = U.ka + 128 * j, nq = min(128, U.kb - q0);
                // this key row over the tile's queries: the queries that attend it are its own family range
                const int jl = max(lo - q0, 0), jh = min(hi - q0, nq);
                const bool has = inb && jh > jl;
                const int c_self = row - q0, c_head = (lo < row) ? lo - q0 : -0x40000000;
                const bool keep_head = (a.dirs & 4) != 0, keep_rest = (a.dirs & ((lo >= row) ? 1 : 2)) != 0;
                uint8_t *ds = sDS + db * 2 * SUB + x * SUB;
                const float2 *stat = sStat + db * 128 + 64 * x + 32 * qh;
                // keep masks of the two 16-query pieces, and what the warp as a whole needs of them
                uint32_t km[2];
                bool any[2], all[2];
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    km[i] = has ? keep_mask<DIRS>(64 * x + 32 * qh + 16 * i, 16, jl, jh, c_self, c_head, keep_head, keep_rest) : 0u;
                    any[i] = __any_sync(0xffffffffu, km[i] != 0u);
                    all[i] = __all_sync(0xffffffffu, km[i] == 0xffffu);
                }
                W_MARK(x, t, 0);
                HDT_WAIT(&stat_full[db], (t >> 1) & 1, 12);                      // the queries' statistics are there
                if (t >= 2) HDT_WAIT(&dq_full[db], ((t >> 1) + 1) & 1, 13);     // dQ of tile t - 2 has read this dS^T buffer
                W_MARK(x, t, 1);
                HDT_WAIT(&sdp_full[x], t & 1, 11);                               // (last: this one ends the chain)
                if (!HDT_AGREE()) break;
                tc_fence_after();
                W_MARK(x, t, 2);
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    uint32_t s_[16], d_[16], pp[8], pd[8];
                    if (any[i]) {
                        tmem_ld16(tm_s + 16u * i, s_);
                        tmem_ld16(tm_dp + 16u * i, d_);
                        tmem_wait_ld();
                    }
                    if (all[i]) {
                        // every key of the warp keeps all 16 queries of the piece: no predicates
#pragma unroll
                        for (int j = 0; j < 16; j += 2) {
                            const float4 st = *reinterpret_cast<const float4 *>(&stat[16 * i + j]);
                            const float p0 = exp2f(fmaf(__uint_as_float(s_[j]), a.scale_log2, -st.x));
                            const float p1 = exp2f(fmaf(__uint_as_float(s_[j + 1]), a.scale_log2, -st.z));
                            pp[j >> 1] = pack_bf16(p0, p1);
                            pd[j >> 1] = pack_bf16(p0 * fmaf(__uint_as_float(d_[j]), a.scale, -st.y), p1 * fmaf(__uint_as_float(d_[j + 1]), a.scale, -st.w));
                        }
                    } else if (any[i] && km[i] != 0u) {
#pragma unroll
                        for (int j = 0; j < 16; j += 2) {
                            const float4 st = *reinterpret_cast<const float4 *>(&stat[16 * i + j]);
                            float p0 = 0.f, p1 = 0.f, e0 = 0.f, e1 = 0.f;
                            if (km[i] & (1u << j)) {
                                p0 = exp2f(fmaf(__uint_as_float(s_[j]), a.scale_log2, -st.x));
                                e0 = p0 * fmaf(__uint_as_float(d_[j]), a.scale, -st.y);
                            }
                            if (km[i] & (2u << j)) {
                                p1 = exp2f(fmaf(__uint_as_float(s_[j + 1]), a.scale_log2, -st.z));
                                e1 = p1 * fmaf(__uint_as_float(d_[j + 1]), a.scale, -st.w);
                            }
                            pp[j >> 1] = pack_bf16(p0, p1);
                            pd[j >> 1] = pack_bf16(e0, e1);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; ++j) { pp[j] = 0u; pd[j] = 0u; }
                    }
                    // P^T: the piece's 16 queries are 8 packed columns, inside the S^T columns this warp has read
                    tmem_st8(tm_s + 8u * i, pp);
                    tmem_st8(tm_dp + 8u * i, pd);      // dS^T for dK, inside the dP^T columns this warp has read
                    *reinterpret_cast<uint4 *>(ds + swz(kl, 4 * qh + 2 * i)) = make_uint4(pd[0], pd[1], pd[2], pd[3]);
                    *reinterpret_cast<uint4 *>(ds + swz(kl, 4 * qh + 2 * i + 1)) = make_uint4(pd[4], pd[5], pd[6], pd[7]);
                }
                tmem_wait_st();
                fence_proxy_async_smem();
                tc_fence_before();
                mbar_arrive(&pds_ready[x]);
                W_MARK(x, t, 3);
                ++t;
                if (j + 1 < nt) ++j;
                else { U = N; N = unit_rec(k++); lo = lo_n; hi = hi_n; j = 0; }
            }
        } else if (warp < W_LOAD) {
            // ================= drain group: the dQ tile of every tile pair, added to the fp32 buffer =================
            const int rl = tid & 127;
            bool go = true;
            for (Walk w = begin(); w.valid && go; step(w)) {
                const WUnit &U = w.U;
                const int t = w.t, db = t & 1;
                W_MARK(2, t, 0);
                // ---- end of a unit: dK and dV of this thread's key row (the next unit's MMAs wait for the
                // accumulators).  bf16 rows staged in the unit's K / V buffer, one swizzled [128 x 64] tile per
                // tensor, TMA stores; the load warp takes the buffer for the unit after the next once the stores have
                // read it.  dV first: its last MMA is the first of the tile's step b, and V's last reader (S^T / dP^T of
                // this tile) was issued a tile ago, so the V half of the buffer is free before the tile's dQ is done;
                // dK, whose half dQ = dS K still reads, after the wait for dQ.  32 columns a round; no factor: the
                // compute warps put softmax_scale into dS. ----
                const bool last = w.j == U.nt - 1;
                const int nrows = U.r1 - U.r0, kvb = w.uc & 1;
                uint8_t *skv = sKV + kvb * 2 * SUB;
                int up = -1;
                if (last && rl < nrows && a.part_dk != nullptr) up = a.up[U.r0 + rl];
                auto round = [&](uint32_t tm_acc, float *part, uint8_t *stage, int c0, uint64_t *read_bar) {
                    uint32_t r[32];
                    tmem_ld32(tm_acc + lane_base + c0, r);
                    tmem_wait_ld();
                    if (read_bar != nullptr) {      // the accumulator has been read: the next unit may overwrite it
                        tc_fence_before();
                        mbar_arrive(read_bar);
                    }
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        if (up >= 0) {      // this row lives on in the next stage: its fp32 gradients go there too
                            float4 *pt = reinterpret_cast<float4 *>(part + ((size_t)up * H + U.h) * D + c0 + j);
                            pt[0] = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
                            pt[1] = make_float4(__uint_as_float(r[j + 4]), __uint_as_float(r[j + 5]), __uint_as_float(r[j + 6]), __uint_as_float(r[j + 7]));
                        }
                        *reinterpret_cast<uint4 *>(stage + swz(rl, (c0 + j) >> 3)) =
                            make_uint4(pack_bf16(__uint_as_float(r[j]), __uint_as_float(r[j + 1])), pack_bf16(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3])),
                                       pack_bf16(__uint_as_float(r[j + 4]), __uint_as_float(r[j + 5])), pack_bf16(__uint_as_float(r[j + 6]), __uint_as_float(r[j + 7])));
                    }
                };
                if (last) {
                    HDT_WAIT(dvacc_full, w.uc & 1, 26);
                    if (HDT_AGREE()) {
                        tc_fence_after();
                        round(tmem + TM_DV, a.part_dv, skv + SUB, 0, nullptr);
                        round(tmem + TM_DV, a.part_dv, skv + SUB, 32, dv_free);
                    }
                }
                HDT_WAIT(&dq_full[db], (t >> 1) & 1, 14);
                W_MARK(2, t, 1);
                if (last) {
                    const int bx = max(__clz(nrows) - 25, 0);
                    const int bbox = 64 >> bx;
                    HDT_WAIT(acc_full, w.uc & 1, 15);
                    if (HDT_AGREE()) {
                        tc_fence_after();
                        round(tmem + TM_DK, a.part_dk, skv, 0, nullptr);
                        round(tmem + TM_DK, a.part_dk, skv, 32, dk_free);
                    }
                    fence_proxy_async_smem();
                    go = group_all(ok, 1, 128);
                    if (!go) break;
                    // rows [0, nrows) of each staged tile as at most two boxes of b rows, b the largest power of two
                    // <= min(nrows, 64): [0, b) and [nrows - b, nrows); where the two overlap the same values are written twice
                    if (rl == 0) {
#pragma unroll
                        for (int tt = 0; tt < 2; ++tt) {
                            tma_store_3d(&sm_out.m[1 + tt][bx], 0, U.h, U.r0, skv + tt * SUB);
                            if (nrows > bbox) tma_store_3d(&sm_out.m[1 + tt][bx], 0, U.h, U.r0 + nrows - bbox, skv + tt * SUB + (nrows - bbox) * 128);
                        }
                        bulk_commit();
                        bulk_wait_read();
                        mbar_arrive(&kv_reuse[kvb]);
                    }
                }
                uint8_t *stg = sStg;
                // fp32 staging: row = query, one swizzled [128 x 32] sub-tile per column half, a TMA reduce-add copy
                // each (requested by the reduce warp).  Rows beyond the span's end hold exact zeros (their dS is zero).
                if (t >= 1) HDT_WAIT(&stg_free[0], (t - 1) & 1, 20);      // the copies of tile t - 1 have read the staging area
                if (!HDT_AGREE()) break;
                tc_fence_after();
#pragma unroll
                for (int half = 0; half < 2; ++half) {      // 32 columns per round of TMEM loads
                    uint32_t r[32];
                    tmem_ld32(tmem + TM_DQ + 64u * db + lane_base + 32u * half, r);
                    tmem_wait_ld();
                    if (half == 1) {          // the accumulator has been read: dQ of tile t + 2 may overwrite it
                        tc_fence_before();
                        mbar_arrive(&dq_free[db]);
                    }
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        *reinterpret_cast<uint4 *>(stg + half * SUB + swz(rl, c)) = make_uint4(r[4 * c], r[4 * c + 1], r[4 * c + 2], r[4 * c + 3]);
                }
                fence_proxy_async_smem();
                mbar_arrive(&stg_full[0]);       // the reduce warp requests the copies
                W_MARK(2, t, 2);
            }
        }
    }
    if (!ok) {
        if (atomicCAS(a.status, 0, HDT_ERR_TIMEOUT) == 0) {
            a.status[1] = (KID << 8) | fail_site;
            a.status[2] = (int)blockIdx.x;
        }
    }
#undef HDT_WAIT
#undef HDT_AGREE
    tc_fence_before();
    __syncthreads();
    if (MARKS && blockIdx.x == 0 && tid < 80) g_bwd_w_marks[tid] = s_marks[tid];
    if (warp == 0) tmem_dealloc(tmem, TM_COLS);
}

int read_bwd_w_marks(long long *out128) {
    HDT_CUDA_CHECK(cudaMemcpyFromSymbol(out128, g_bwd_w_marks, sizeof(long long) * 128));
    return HDT_OK;
}
int read_bwd_w_tiles(long long *out512) {
    HDT_CUDA_CHECK(cudaMemcpyFromSymbol(out512, g_bwd_w_tiles, sizeof(long long) * 512));
    return HDT_OK;
}

int launch_bwd_tc_onewalk64(const BwdStageArgs &a, const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv,
                            const CUtensorMap &tdo, const StoreMaps &outs, const CUtensorMap &tacc, int n_empty, cudaStream_t st) {
    constexpr int smem_max = 14 * SUB + 2 * 1024 + 256 + 640;
    const int smem = smem_max - ((a.phases == 86 && a.dirs == 7) ? 0 : 640);      // (the clock marks of an instrumented run)
    static DevOnce attr;
    if (!attr.done()) {
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc_w<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max));
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc_w<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max));
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc_w<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max));
        attr.set();
    }
    int n_sm = 0;
    if (const int rc = sm_count(&n_sm)) return rc;
    const int n_rest = a.nb - a.n_fused;
    if (n_rest <= 0) return HDT_OK;
    if (a.delta == nullptr || a.dq_acc == nullptr || n_empty < 0 || n_empty != a.n_empty)
        return set_error(HDT_ERR_INVALID_ARG, "launch_bwd_tc_onewalk64: needs delta, the fp32 dQ buffer and the number of EMPTY blocks");
    const long long units = (long long)n_rest * a.H;
    const int grid = (int)(units < n_sm ? units : n_sm);
    if (a.phases == 86 && a.dirs == 7) k_bwd_tc_w<false, true><<<grid, 736, smem, st>>>(tq, tk, tv, tdo, outs, tacc, a);
    else if (a.dirs != 7) k_bwd_tc_w<true><<<grid, 736, smem, st>>>(tq, tk, tv, tdo, outs, tacc, a);
    else k_bwd_tc_w<false><<<grid, 736, smem, st>>>(tq, tk, tv, tdo, outs, tacc, a);
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;      // (the EMPTY blocks, the last n_empty of queue_split, get their zero rows from k_dq_finish)
}

}  // namespace hdt
