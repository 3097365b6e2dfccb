// Transposed looping backward for stage 0 in bf16 at D = 64: SELF, non-EMPTY blocks (both tiles of
// the pass are the block itself).
//
// The tile pass of hdt_attn_tc_bwd.cu with keys in the TMEM lanes instead of queries:
//   MMA   S^T = K Q^T, dP^T = V dO^T                                  -> TMEM (lane = key)
//   keys  P^T = exp2(S^T c - LSE[query]) on the queries inside the key's family range (the ranges
//         of a stage are symmetric: the queries that attend key j are j's own range),
//         dS^T = P^T o (dP^T - delta[query]);
//         P^T (bf16) stays in TMEM, over the S^T columns it was computed from; dS^T -> shared memory
//   MMA   dV = P^T dO with the A operand read from TMEM; dK = dS^T Q and dQ = dS K with dS^T from
//         shared memory (K-major for dK, MN-major for dQ)            -> TMEM
// Only dS^T needs a shared-memory tile, so a CTA takes 112 KB of shared memory and 256 TMEM columns
// and two CTAs share an SM: while one waits for its loads or MMAs, drains or stores, the other
// computes.  Each CTA stays resident and walks the items blockIdx.x, + gridDim.x, ... of
// queue_split x heads; the next item's four input tiles are requested as soon as the output MMAs
// of the current one have finished.
// Thread t: TMEM lane t % 128 (a key row; for dQ a query row), column half t / 128.
#include <cuda_bf16.h>

#include "hdt_internal.cuh"
#include "hdt_sm100.cuh"
#include "hdt_tmap.cuh"

namespace hdt {
using namespace sm100;

namespace {
constexpr int SUB = 16384;
constexpr long long WAIT_CYCLES = 400000000LL;
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

// 16 bytes read once: not kept in L1 (which shares its storage with the tiles in shared memory)
__device__ __forceinline__ uint4 ld_stream(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
}  // namespace

// TMEM columns.  S^T occupies 0..127 and dP^T 128..255 until the keys have turned them into P^T and
// dS^T.  The column half hf = 0 (queries 0..63) packs its P^T over columns 0..31, hf = 1 (queries
// 64..127) over columns 96..127: every thread overwrites only columns that it alone reads and has
// already read (hf = 1 takes its two slices in descending order).  That leaves 32..95 for dV; dK and
// dQ go over the dead dP^T columns.
// STAMP: thread 0 of CTA 0 adds the cycles of each phase of its item loop to g_bwd_t_phase_cycles (diagnostics).
__device__ long long g_bwd_t_phase_cycles[16];
__device__ long long g_bwd_t_timeline[512][4];   // STAMP: per CTA: globaltimer at entry, first tiles in, loop end; SM id
__device__ __forceinline__ long long gtime() { long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
#define HDT_TSTAMP(i)                                                              \
    do {                                                                           \
        if constexpr (STAMP) {                                                     \
            if (tid == 0 && blockIdx.x == 0) {                                     \
                const long long now_ = clock64();                                  \
                atomicAdd((unsigned long long *)&g_bwd_t_phase_cycles[i], (unsigned long long)(now_ - t_last)); \
                t_last = now_;                                                     \
            }                                                                      \
        }                                                                          \
    } while (0)

// FD (fused delta): a.delta is not read; delta[query] = dO[query] . O[query] is computed here: eight
// lanes per token row, 16 bytes each of O and dO, requested at the top of the item (past L1) and
// reduced once S^T and dP^T are there.  (dO from its tile in shared memory instead: 8 % slower.)
template <bool DIRS, bool STAMP = false, bool FD = false>
__global__ void __maxnreg__(120) k_bwd_tc_t(const __grid_constant__ CUtensorMap tm_q,
                                                     const __grid_constant__ CUtensorMap tm_k,
                                                     const __grid_constant__ CUtensorMap tm_v,
                                                     const __grid_constant__ CUtensorMap tm_do,
                                                     const __grid_constant__ StoreMaps sm_out, const BwdStageArgs a) {
    constexpr int D = 64;
    constexpr uint32_t TM_S = 0, TM_DP = 128, TM_DV = 32, TM_DK = 128, TM_DQ = 192, TM_COLS = 256;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *sQ = smem_raw, *sDO = sQ + SUB, *sK = sDO + SUB, *sV = sK + SUB;
    uint8_t *sDS = sV + SUB;              // dS^T: sub-tile u = queries 64u..64u+63, row = key; later staging of dQ, dK
    uint8_t *sStg = sDS + 2 * SUB;        // staging of dV
    uint64_t *bar_in = (uint64_t *)(sStg + SUB);
    uint64_t *bar_a = bar_in + 1, *bar_b = bar_in + 2;
    uint32_t *slot = (uint32_t *)(bar_in + 3);
    volatile int *abort_flag = (volatile int *)(slot + 1);
    float2 *sStat = (float2 *)sV;         // LSE, delta of the item's queries; V is dead once dP^T is there

    const int tid = threadIdx.x, warp = tid >> 5, rl = tid & 127, hf = tid >> 7;
    if constexpr (STAMP) { if (tid == 0 && blockIdx.x < 512) { g_bwd_t_timeline[blockIdx.x][0] = gtime(); unsigned sm; asm("mov.u32 %0, %%smid;" : "=r"(sm)); g_bwd_t_timeline[blockIdx.x][3] = sm; } }
    const int H = a.H, G = gridDim.x;
    const float LOG2E = 1.4426950408889634f;
    const int n_items = a.n_fused * H;

    if ((smem_u32(smem_raw) & 1023u) != 0u) {      // the swizzled tiles need 1024-byte alignment
        if (tid == 0) atomicCAS(a.status, 0, HDT_ERR_CUDA);
        return;
    }
    // Item i of this CTA is entry blockIdx.x + i * G of queue_split x heads.  Its block number is
    // read three items ahead and its record two items ahead, so that no load in the loop waits for
    // another one.
    struct It { int valid, r0, r1, h; };
    auto block_of = [&](int i) { return i < n_items ? a.queue_split[i / H] : -1; };
    auto fetch = [&](int i, int blk) {
        It x{0, 0, 0, 0};
        if (blk >= 0) {
            const int *rec = a.blocks + 5 * (size_t)blk;
            x.valid = 1; x.r0 = rec[0]; x.r1 = rec[1]; x.h = i % H;
        }
        return x;
    };
    auto issue_loads = [&](const It &d) {       // thread 0
        mbar_expect_tx(bar_in, 4u * SUB);
        tma_load_3d(sK, &tm_k, 0, d.h, d.r0, bar_in);
        tma_load_3d(sQ, &tm_q, 0, d.h, d.r0, bar_in);
        tma_load_3d(sV, &tm_v, 0, d.h, d.r0, bar_in);
        tma_load_3d(sDO, &tm_do, 0, d.h, d.r0, bar_in);
    };
    if (tid == 0) {
        mbar_init(bar_in, 1);
        mbar_init(bar_a, 2);
        mbar_init(bar_b, 3);
        fence_mbar_init();
        // the first item's tiles are requested before anything else is set up
        if ((int)blockIdx.x < n_items) issue_loads(fetch((int)blockIdx.x, block_of((int)blockIdx.x)));
        *abort_flag = (*a.status != 0);
    }
    if (warp == 0) tmem_alloc(slot, TM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *slot;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const bool dead = (*abort_flag != 0);
    bool ok = true;
    const bool issuer = ((tid & 31) == 0) && warp < 3;
    const bool store_thread = ((tid & 31) == 0) && warp >= 2;     // six threads: two boxes per gradient tensor

    struct RowStat { int lo, hi, up; float lse, dl; };
    auto load_stat = [&](const It &d) {
        RowStat r{0, 0, -1, 0.f, 0.f};
        const int row = d.r0 + rl;
        if (d.valid && row < d.r1) {
            r.lo = a.rng[2 * row];
            r.hi = a.rng[2 * row + 1];
            r.lse = a.lse[(size_t)d.h * a.T + row];
            if constexpr (!FD) r.dl = a.delta[(size_t)d.h * a.T + row];
            if (a.part_dq != nullptr) r.up = a.up[row];
        }
        return r;
    };

    if (!dead && n_items > 0) {
        const int i0 = (int)blockIdx.x;
        It d0 = fetch(i0, block_of(i0)), d1 = fetch(i0 + G, block_of(i0 + G));
        int b2 = block_of(i0 + 2 * G);
        RowStat rc = load_stat(d0);
        long long t_last = STAMP ? clock64() : 0;
        for (int it = 0; d0.valid && !*abort_flag; ++it) {
            const int r0 = d0.r0, r1 = d0.r1, h = d0.h, nrows = r1 - r0;
            const int Nc = (nrows + 15) & ~15;
            uint4 xo[4], xg[4];      // FD: chunk tid % 8 of rows tid / 8 + 32 k of O and dO
            if constexpr (FD) {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int r = (tid >> 3) + 32 * k;
                    xo[k] = make_uint4(0u, 0u, 0u, 0u);
                    xg[k] = make_uint4(0u, 0u, 0u, 0u);
                    if (r < nrows) {
                        const size_t off = ((size_t)(r0 + r) * H + h) * D + (tid & 7) * 8;
                        xo[k] = ld_stream(reinterpret_cast<const __nv_bfloat16 *>(a.o) + off);
                        xg[k] = ld_stream(reinterpret_cast<const __nv_bfloat16 *>(a.d_o) + off);
                    }
                }
            }
            // the next item's tiles start their way from HBM to L2 now; the loads into shared memory
            // (requested once this item's output MMAs have released the tiles) then find them there
            if (tid == 0 && d1.valid) {
                tma_prefetch_3d(&tm_k, 0, d1.h, d1.r0);
                tma_prefetch_3d(&tm_q, 0, d1.h, d1.r0);
                tma_prefetch_3d(&tm_v, 0, d1.h, d1.r0);
                tma_prefetch_3d(&tm_do, 0, d1.h, d1.r0);
            }
            HDT_TSTAMP(0);
            ok = mbar_wait(bar_in, it & 1, abort_flag, WAIT_CYCLES) && ok;
            HDT_TSTAMP(1);
            if constexpr (STAMP) { if (tid == 0 && it == 0 && blockIdx.x < 512) g_bwd_t_timeline[blockIdx.x][1] = gtime(); }
            if (issuer && warp < 2 && !*abort_flag) {      // warp 0: S^T = K Q^T, warp 1: dP^T = V dO^T
                tc_fence_after();
                const uint32_t idesc = idesc_bf16(Nc, false, false);
                const uint32_t sa = smem_u32(warp == 0 ? sK : sV), sb = smem_u32(warp == 0 ? sQ : sDO);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk)
                    mma_ss(tmem + (warp == 0 ? TM_S : TM_DP), smem_desc(sa + kk * 32, 0, 1024), smem_desc(sb + kk * 32, 0, 1024),
                           idesc, kk > 0);
                mma_commit(bar_a);
            }
            const bool inq = rl < nrows;
            // this row as a key: the queries that attend it are its own family range
            const int jl = max(rc.lo - r0, 0), jh = min(rc.hi - r0, nrows);
            const bool has = inq && jh > jl;
            const int e_row = r0 + rl;
            const int c_self = rl, c_head = (rc.lo < e_row) ? rc.lo - r0 : -0x40000000;
            // entry (query, key = this row): the query is this row's parent (parent -> child, bit 4),
            // one of its children (child -> parent, bit 1) or a sibling (bit 2)
            const bool keep_head = (a.dirs & 4) != 0, keep_rest = (a.dirs & ((rc.lo >= e_row) ? 1 : 2)) != 0;
            HDT_TSTAMP(2);
            ok = mbar_wait(bar_a, it & 1, abort_flag, WAIT_CYCLES) && ok;
            // this row as a query: its statistics for the key threads, over the V tile
            if constexpr (FD) {
                if (hf == 0) sStat[rl].x = rc.lse * LOG2E;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t xs[4] = {xo[k].x, xo[k].y, xo[k].z, xo[k].w}, ys[4] = {xg[k].x, xg[k].y, xg[k].z, xg[k].w};
                    float acc = 0.f;
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        acc = fmaf(__uint_as_float(xs[w] << 16), __uint_as_float(ys[w] << 16), acc);
                        acc = fmaf(__uint_as_float(xs[w] & 0xffff0000u), __uint_as_float(ys[w] & 0xffff0000u), acc);
                    }
                    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
                    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
                    acc += __shfl_xor_sync(0xffffffffu, acc, 4);
                    if ((tid & 7) == 0) sStat[(tid >> 3) + 32 * k].y = acc;
                }
            } else {
                if (hf == 0) sStat[rl] = make_float2(rc.lse * LOG2E, rc.dl);
            }
            if (store_thread) bulk_wait_read();            // the previous item's staged gradients have left shared memory
            __syncthreads();
            tc_fence_after();
            HDT_TSTAMP(3);
#pragma unroll
            for (int step = 0; step < 2; ++step) {
                const int sl = hf ? 1 - step : step;       // hf = 1: descending (see the column map above)
                const int s0 = 64 * hf + 32 * sl;
                if (s0 >= Nc) continue;                    // same decision in the whole warp
                const uint32_t km = has ? keep_mask<DIRS>(s0, 32, jl, jh, c_self, c_head, keep_head, keep_rest) : 0u;
                const bool mine = km != 0u;
                uint32_t pp[16], pd[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) { pp[j] = 0u; pd[j] = 0u; }
                if (__any_sync(0xffffffffu, mine)) {
                    uint32_t rs[32], rd[32];
                    tmem_ld32(tmem + TM_S + lane_base + s0, rs);
                    tmem_ld32(tmem + TM_DP + lane_base + s0, rd);
                    tmem_wait_ld();
                    if (mine) {
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            const float4 st = *reinterpret_cast<const float4 *>(&sStat[s0 + j]);   // lse2, delta of two queries
                            float p0 = 0.f, p1 = 0.f, e0 = 0.f, e1 = 0.f;
                            if (km & (1u << j)) {
                                p0 = exp2f(fmaf(__uint_as_float(rs[j]), a.scale_log2, -st.x));
                                e0 = p0 * (__uint_as_float(rd[j]) - st.y);
                            }
                            if (km & (2u << j)) {
                                p1 = exp2f(fmaf(__uint_as_float(rs[j + 1]), a.scale_log2, -st.z));
                                e1 = p1 * (__uint_as_float(rd[j + 1]) - st.w);
                            }
                            pp[j >> 1] = pack_bf16(p0, p1);
                            pd[j >> 1] = pack_bf16(e0, e1);
                        }
                    }
                }
                // P^T: queries s0..s0+31 are K indices s0..s0+31 of the dV MMA = 16 packed columns
                tmem_st16(tmem + lane_base + (hf ? 96u : 0u) + 16u * sl, pp);
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    *reinterpret_cast<uint4 *>(sDS + hf * SUB + swz(rl, sl * 4 + c)) =
                        make_uint4(pd[4 * c], pd[4 * c + 1], pd[4 * c + 2], pd[4 * c + 3]);
            }
            tmem_wait_st();
            fence_proxy_async_smem();
            tc_fence_before();
            HDT_TSTAMP(4);
            __syncthreads();
            HDT_TSTAMP(5);
            if (issuer && !*abort_flag) {
                tc_fence_after();
                if (warp == 0) {            // dV = P^T dO: A from TMEM, B = dO (MN-major)
                    const uint32_t idesc = idesc_bf16(D, false, true);
                    for (int kk = 0; kk < Nc / 16; ++kk)
                        mma_ts(tmem + TM_DV, tmem + (kk < 4 ? 8u * kk : 96u + 8u * (kk - 4)),
                               smem_desc(smem_u32(sDO) + kk * 2048, SUB, 1024), idesc, kk > 0);
                } else if (warp == 1) {     // dK = dS^T Q: A = dS^T (K-major), B = Q (MN-major)
                    const uint32_t idesc = idesc_bf16(D, false, true);
                    for (int kk = 0; kk < Nc / 16; ++kk)
                        mma_ss(tmem + TM_DK, smem_desc(smem_u32(sDS) + (kk / 4) * SUB + (kk % 4) * 32, 0, 1024),
                               smem_desc(smem_u32(sQ) + kk * 2048, SUB, 1024), idesc, kk > 0);
                } else {                    // dQ = dS K: A = dS (MN-major: stored as dS^T), B = K (MN-major)
                    const uint32_t idesc = idesc_bf16(D, true, true);
                    for (int kk = 0; kk < Nc / 16; ++kk)
                        mma_ss(tmem + TM_DQ, smem_desc(smem_u32(sDS) + kk * 2048, SUB, 1024),
                               smem_desc(smem_u32(sK) + kk * 2048, SUB, 1024), idesc, kk > 0);
                }
                mma_commit(bar_b);
            }
            HDT_TSTAMP(6);
            // prefetch while the output MMAs run
            const It d2 = fetch(i0 + (it + 2) * G, b2);                // record two items ahead
            const int b3 = block_of(i0 + (it + 3) * G);                // block number three items ahead
            HDT_TSTAMP(13);
            const RowStat rn = load_stat(d1);                          // row statistics one item ahead
            HDT_TSTAMP(14);
            ok = mbar_wait(bar_b, it & 1, abort_flag, WAIT_CYCLES) && ok;
            tc_fence_after();
            HDT_TSTAMP(7);
            // the input tiles are free: the next item's loads fly during the drain and the stores
            if (tid == 0 && d1.valid && !*abort_flag) issue_loads(d1);
            // ---- drain: this thread's row, its half of the D columns of each gradient ----
            {
                const uint32_t cols[3] = {TM_DQ, TM_DK, TM_DV};
                uint8_t *dsts[3] = {sDS, sDS + SUB, sStg};
                float *parts[3] = {a.part_dq, a.part_dk, a.part_dv};
#pragma unroll
                for (int t = 0; t < 3; ++t) {
                    const float sc = (t == 2) ? 1.f : a.scale;
                    float *part = (inq && rc.up >= 0) ? parts[t] + ((size_t)rc.up * H + h) * D : nullptr;
                    const int c0 = hf * 32;
                    uint32_t r[32];
                    tmem_ld32(tmem + cols[t] + lane_base + c0, r);
                    tmem_wait_ld();
                    uint32_t pk[16];
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const float x0 = __uint_as_float(r[j]) * sc, x1 = __uint_as_float(r[j + 1]) * sc;
                        const float x2 = __uint_as_float(r[j + 2]) * sc, x3 = __uint_as_float(r[j + 3]) * sc;
                        if (part != nullptr) *reinterpret_cast<float4 *>(part + c0 + j) = make_float4(x0, x1, x2, x3);
                        pk[j >> 1] = pack_bf16(x0, x1);
                        pk[(j >> 1) + 1] = pack_bf16(x2, x3);
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        *reinterpret_cast<uint4 *>(dsts[t] + swz(rl, (c0 >> 3) + c)) =
                            make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                }
            }
            HDT_TSTAMP(8);
            fence_proxy_async_smem();
            tc_fence_before();
            __syncthreads();
            HDT_TSTAMP(9);
            // ---- TMA stores: rows [0, nrows) of each staged tile as at most two boxes of b rows, b the
            // largest power of two <= min(nrows, 64): [0, b) and [nrows - b, nrows); where the two
            // overlap the same values are written twice.  They read shared memory until the next
            // item's key threads are about to overwrite it. ----
            if (store_thread) {
                const int t = (warp - 2) >> 1, second = (warp - 2) & 1;
                const int bx = max(__clz(nrows) - 25, 0);          // box of 64 >> bx rows: 64 for nrows >= 64
                const int b = 64 >> bx;
                const int off = second ? nrows - b : 0;
                if (!second || nrows > b) tma_store_3d(&sm_out.m[t][bx], 0, h, r0 + off, (t == 2 ? sStg : sDS + t * SUB) + off * 128);
                bulk_commit();
            }
            HDT_TSTAMP(10);
            HDT_TSTAMP(11);
            if constexpr (STAMP) { if (tid == 0 && blockIdx.x == 0) atomicAdd((unsigned long long *)&g_bwd_t_phase_cycles[12], 1ull); }
            d0 = d1; d1 = d2; rc = rn; b2 = b3;
        }
    }
    if (dead && (int)blockIdx.x < n_items) {     // an earlier failure: only let the tiles requested above land
        volatile int none = 0;
        (void)mbar_wait(bar_in, 0, &none, WAIT_CYCLES);
    }
    if (!ok && tid == 0) atomicCAS(a.status, 0, HDT_ERR_TIMEOUT);
    if (store_thread) bulk_wait_read();
    if constexpr (STAMP) { if (tid == 0 && blockIdx.x < 512) g_bwd_t_timeline[blockIdx.x][2] = gtime(); }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TM_COLS);
}

int launch_bwd_tc_fused64(const BwdStageArgs &a, const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv,
                          const CUtensorMap &tdo, const StoreMaps &outs, cudaStream_t st) {
    constexpr int smem = 7 * SUB + 64;
    static DevOnce attr;
    int n_sm = 0;
    if (const int rc_ = sm_count(&n_sm)) return rc_;
    if (!attr.done()) {
        const void *fns[6] = {(const void *)k_bwd_tc_t<false>,       (const void *)k_bwd_tc_t<true>,
                              (const void *)k_bwd_tc_t<false, false, true>,
#ifdef HDT_WORKBENCH      // the instrumented instantiations (option "phase_stamps" = 1)
                              (const void *)k_bwd_tc_t<false, true>, (const void *)k_bwd_tc_t<false, true, true>,
#endif
                              nullptr};
        for (int i = 0; fns[i]; ++i) {
            HDT_CUDA_CHECK(cudaFuncSetAttribute(fns[i], cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            HDT_CUDA_CHECK(cudaFuncSetAttribute(fns[i], cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
        }
        attr.set();
    }
    const long long items = (long long)a.n_fused * a.H;
    if (items == 0) return HDT_OK;
    const bool fd = a.delta == nullptr;
    if (fd && (a.o == nullptr || a.dirs != 7))
        return set_error(HDT_ERR_INVALID_ARG, "launch_bwd_tc_fused64: the fused-delta kernel needs o and the full rule");
    const long long slots = (a.no_persistent == 6 ? 1LL : 2LL) * n_sm;
    const int grid = (int)(items < slots ? items : slots);
#ifdef HDT_WORKBENCH
    if (g_phase_stamps == 1 && a.dirs == 7) {
        if (fd) k_bwd_tc_t<false, true, true><<<grid, 256, smem, st>>>(tq, tk, tv, tdo, outs, a);
        else k_bwd_tc_t<false, true><<<grid, 256, smem, st>>>(tq, tk, tv, tdo, outs, a);
    } else
#endif
    if (a.dirs != 7) k_bwd_tc_t<true><<<grid, 256, smem, st>>>(tq, tk, tv, tdo, outs, a);
    else if (fd) k_bwd_tc_t<false, false, true><<<grid, 256, smem, st>>>(tq, tk, tv, tdo, outs, a);
    else k_bwd_tc_t<false><<<grid, 256, smem, st>>>(tq, tk, tv, tdo, outs, a);
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;
}

// Diagnostics: cycles CTA 0 spent per phase since the last call (12 phases, then the item count),
// added to out16; resets the counters.
int read_bwd_t_phase_cycles(long long *out16) {
    long long v[16];
    HDT_CUDA_CHECK(cudaMemcpyFromSymbol(v, g_bwd_t_phase_cycles, sizeof(v)));
    for (int i = 0; i < 16; ++i) out16[i] += v[i];
    long long zero[16] = {0};
    HDT_CUDA_CHECK(cudaMemcpyToSymbol(g_bwd_t_phase_cycles, zero, sizeof(zero)));
    return HDT_OK;
}

int read_bwd_t_timeline(long long *out2048) {
    HDT_CUDA_CHECK(cudaMemcpyFromSymbol(out2048, g_bwd_t_timeline, sizeof(long long) * 2048));
    return HDT_OK;
}

}  // namespace hdt
