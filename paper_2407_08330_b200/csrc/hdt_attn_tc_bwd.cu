// Tensor-core backward for stage 0 in bf16 (TMA + tcgen05/TMEM).
//
// One CTA (256 threads) per (row block, head).  A "tile pass" takes a query-side tile (Q, dO of
// 128 token rows with their LSE and delta) and a key-side tile (K, V of 128 token rows):
//   MMA   S = Q K^T, dP = dO V^T                                   -> TMEM
//   rows  P = exp2(S*c - LSE) on the columns inside the row's family range, dS = P o (dP - delta);
//         P and dS (bf16) -> shared memory, one sub-tile per 64 keys
//   MMA   dQ += dS K  |  dV += P^T dO, dK += dS^T Q                 -> TMEM
// Thread t handles row t % 128 (its TMEM lane) and the column half t / 128.
// A block whose key span lies inside its own rows (the usual case: blocks are packed from whole
// families) needs one pass with both tiles equal to the block; at D = 64 that pass produces dQ,
// dK and dV together (5 MMAs).  Otherwise the block first walks its key span as a query block
// (dQ), then walks the same span as a key block (dK, dV); the family ranges are symmetric, so the
// same index serves both.
#include <cuda_bf16.h>

#include "hdt_internal.cuh"
#include "hdt_sm100.cuh"
#include "hdt_tmap.cuh"

namespace hdt {
using namespace sm100;

static constexpr int SUB = 16384;
static constexpr long long WAIT_CYCLES = 400000000LL;
__device__ __forceinline__ uint32_t swz(int r, int c) { return (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4)); }

// Stages above 0: elements [row0, row0 + 128) of the stage are token rows tok[e] of [T, H, D] bf16
// tensors.  The threads copy them (head h) into D / 64 swizzled sub-tiles per tensor, the layout
// the TMA loads of stage 0 produce; elements at or beyond `end` become zero rows.  Thread t owns
// 16-byte chunk t % 8 of rows t / 8, t / 8 + NT / 8, ...; all indices are loaded first, then all
// rows of all NTEN tensors, then everything is stored, so that the loads overlap.
template <int D, int NT, int NTEN>
__device__ __forceinline__ void gather_tiles(uint8_t *const (&dst)[NTEN], const void *const (&src)[NTEN],
                                             const int *__restrict__ tok, int row0, int end, int H, int h, int tid) {
    constexpr int RPP = NT / 8, NP = 128 / RPP, NSUB = D / 64;
    const int c = tid & 7, rr = tid >> 3;
    int tk[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) {
        const int e = row0 + rr + p * RPP;
        tk[p] = e < end ? tok[e] : -1;
    }
#pragma unroll
    for (int t = 0; t < NSUB; ++t) {
        uint4 v[NTEN][NP];
#pragma unroll
        for (int x = 0; x < NTEN; ++x) {
            const __nv_bfloat16 *g = reinterpret_cast<const __nv_bfloat16 *>(src[x]);
#pragma unroll
            for (int p = 0; p < NP; ++p) {
                v[x][p] = make_uint4(0u, 0u, 0u, 0u);
                if (tk[p] >= 0) v[x][p] = *reinterpret_cast<const uint4 *>(g + ((size_t)tk[p] * H + h) * D + t * 64 + c * 8);
            }
        }
#pragma unroll
        for (int x = 0; x < NTEN; ++x)
#pragma unroll
            for (int p = 0; p < NP; ++p) *reinterpret_cast<uint4 *>(dst[x] + t * SUB + swz(rr + p * RPP, c)) = v[x][p];
    }
}

// The same with delta = dO . O of every gathered row computed on the way (no delta pass ran): src[IDO]
// is dO; the eight lanes that hold a row's chunks also fetch the chunks of its O row, multiply and
// reduce, and lane 0 of the eight leaves the sum in s_delta[row - row0] (0 for rows at or beyond end).
template <int D, int NT, int NTEN, int IDO>
__device__ __forceinline__ void gather_tiles_delta(uint8_t *const (&dst)[NTEN], const void *const (&src)[NTEN], const void *o_rows,
                                                   float *s_delta, const int *__restrict__ tok, int row0, int end, int H, int h,
                                                   int tid) {
    constexpr int RPP = NT / 8, NP = 128 / RPP, NSUB = D / 64;
    const int c = tid & 7, rr = tid >> 3;
    int tk[NP];
    float acc[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) {
        const int e = row0 + rr + p * RPP;
        tk[p] = e < end ? tok[e] : -1;
        acc[p] = 0.f;
    }
#pragma unroll
    for (int t = 0; t < NSUB; ++t) {
        uint4 v[NTEN][NP], vo[NP];
#pragma unroll
        for (int p = 0; p < NP; ++p) {
            vo[p] = make_uint4(0u, 0u, 0u, 0u);
            if (tk[p] >= 0)
                vo[p] = *reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(o_rows) + ((size_t)tk[p] * H + h) * D + t * 64 + c * 8);
        }
#pragma unroll
        for (int x = 0; x < NTEN; ++x) {
            const __nv_bfloat16 *g = reinterpret_cast<const __nv_bfloat16 *>(src[x]);
#pragma unroll
            for (int p = 0; p < NP; ++p) {
                v[x][p] = make_uint4(0u, 0u, 0u, 0u);
                if (tk[p] >= 0) v[x][p] = *reinterpret_cast<const uint4 *>(g + ((size_t)tk[p] * H + h) * D + t * 64 + c * 8);
            }
        }
#pragma unroll
        for (int x = 0; x < NTEN; ++x)
#pragma unroll
            for (int p = 0; p < NP; ++p) *reinterpret_cast<uint4 *>(dst[x] + t * SUB + swz(rr + p * RPP, c)) = v[x][p];
#pragma unroll
        for (int p = 0; p < NP; ++p) {
            const uint32_t xs[4] = {vo[p].x, vo[p].y, vo[p].z, vo[p].w}, ys[4] = {v[IDO][p].x, v[IDO][p].y, v[IDO][p].z, v[IDO][p].w};
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                acc[p] = fmaf(__uint_as_float(xs[w] << 16), __uint_as_float(ys[w] << 16), acc[p]);
                acc[p] = fmaf(__uint_as_float(xs[w] & 0xffff0000u), __uint_as_float(ys[w] & 0xffff0000u), acc[p]);
            }
        }
    }
#pragma unroll
    for (int p = 0; p < NP; ++p) {
        float x = acc[p];
        x += __shfl_xor_sync(0xffffffffu, x, 1);
        x += __shfl_xor_sync(0xffffffffu, x, 2);
        x += __shfl_xor_sync(0xffffffffu, x, 4);
        if (c == 0) s_delta[rr + p * RPP] = x;
    }
}

// GATHER = true: a stage above 0 computed beside stage 0.  Rows (and their LSE / delta) are fetched
// through the stage's tok map by the threads instead of TMA, and the kernel leaves only the stage's
// own gradients per element (fp32, indexed by element) for the chain merge.
// DIRS = true: the index carries direction bits other than 7; entries of the row range that the
// bits switch off are masked as well (dir_ok).
template <int D, bool GATHER = false, bool DIRS = false>
__global__ void __launch_bounds__(256) k_bwd_tc(const __grid_constant__ CUtensorMap tm_q,
                                                const __grid_constant__ CUtensorMap tm_k,
                                                const __grid_constant__ CUtensorMap tm_v,
                                                const __grid_constant__ CUtensorMap tm_do, const BwdStageArgs a) {
    constexpr int NSUB = D / 64;
    // TMEM columns: S and dP per pass (0..255); accumulators.  D = 64: dQ 256, dK 320, dV 384.
    // D = 128 (3 x 128 accumulator columns do not fit beside S and dP): a fused pass puts dV and dK
    // over S and dP, which are dead once P and dS are written; the two-walk path keeps dQ, then
    // dK, in columns 256.. and dV in 384.. while S and dP are rewritten per chunk.
    constexpr uint32_t TM_S = 0, TM_DP = 128, TM_DQ = 256, TM_COLS = 512;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = sm, *sDO = sQ + NSUB * SUB, *sK = sDO + NSUB * SUB, *sV = sK + NSUB * SUB;
    uint8_t *sP = sV + NSUB * SUB, *sDS = sP + 2 * SUB;
    uint64_t *bar_tma = (uint64_t *)(sDS + 2 * SUB);
    uint64_t *bar_mma = bar_tma + 1;
    uint32_t *slot = (uint32_t *)(bar_mma + 1);
    volatile int *abort_flag = (volatile int *)(slot + 1);
    float *s_delta = (float *)(bar_tma + 8);     // gathering kernel without a delta pass: dO . O of the query-side rows

    const int tid = threadIdx.x, warp = tid >> 5, rl = tid & 127, hf = tid >> 7;
    // rest_only: take the blocks after the first n_fused entries of queue_split
    const int blk = a.rest_only ? a.queue_split[a.n_fused + blockIdx.x] : a.queue[blockIdx.x];
    const int h = blockIdx.y, H = a.H;
    const int *rec = a.blocks + 5 * (size_t)blk;
    const int r0 = rec[0], r1 = rec[1], ka = rec[2], kb = rec[3], fl = rec[4];
    const int nrows = r1 - r0;
    const float LOG2E = 1.4426950408889634f;

    if (tid == 0) {
        mbar_init(bar_tma, 1);
        mbar_init(bar_mma, 1);
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
    const bool empty = (fl & HDT_BLK_EMPTY) != 0;
    const bool self = (fl & HDT_BLK_SELF) != 0;
    const bool fused = self && !empty && !dead;   // one pass yields dQ, dK and dV
    const uint32_t TM_DK = (D == 64) ? 320u : (fused ? 128u : 256u);
    const uint32_t TM_DV = (D == 64) ? 384u : (fused ? 0u : 384u);
    uint32_t ph_tma = 0, ph_mma = 0;
    bool ok = true;

    // One tile pass.  q_row0 / k_row0: first token row of the query-side / key-side tile;
    // q_end / k_end: end of the valid rows of each side.
    auto tile_pass = [&](int q_row0, int q_end, int k_row0, int k_end, bool want_dq, bool want_dkdv, bool acc_q,
                         bool acc_kv) {
        const int nq = min(128, q_end - q_row0), nk = min(128, k_end - k_row0);
        const int Nc = (nk + 15) & ~15, Kr = (nq + 15) & ~15;
        if (tid == 0 && !*abort_flag) {
            tc_fence_after();
            const uint32_t idesc = idesc_bf16(Nc, false, false);
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t off = (kk / 4) * SUB + (kk % 4) * 32;
                mma_ss(tmem + TM_S, smem_desc(smem_u32(sQ) + off, 0, 1024), smem_desc(smem_u32(sK) + off, 0, 1024), idesc,
                       kk > 0);
            }
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t off = (kk / 4) * SUB + (kk % 4) * 32;
                mma_ss(tmem + TM_DP, smem_desc(smem_u32(sDO) + off, 0, 1024), smem_desc(smem_u32(sV) + off, 0, 1024), idesc,
                       kk > 0);
            }
            mma_commit(bar_mma);
        }
        // row statistics of this thread's query-side row while the MMAs run
        const int e = q_row0 + rl;
        const bool inq = e < q_end;
        int lo = 0, hi = 0;
        float lse2 = 0.f, dl = 0.f;
        if (inq) {
            lo = a.rng[2 * e];
            hi = a.rng[2 * e + 1];
            if (hi > lo) {
                const int tk = GATHER ? a.tok[e] : e;
                lse2 = a.lse[(size_t)h * a.T + tk] * LOG2E;
                if (a.delta != nullptr) dl = a.delta[(size_t)h * a.T + tk];
                else dl = s_delta[rl];      // no delta pass ran: left by the gather of the query-side rows
            }
        }
        const int jl = max(lo - k_row0, 0), jh = min(hi - k_row0, nk);
        const bool has = inq && jh > jl;
        // direction bits: column of the row itself, of its parent (none for a head row), and
        // whether the parent entry / every other entry of the range is kept
        const int c_self = e - k_row0, c_head = (lo < e) ? lo - k_row0 : -0x40000000;
        const bool keep_head = (a.dirs & 1) != 0, keep_rest = (a.dirs & ((lo >= e) ? 4 : 2)) != 0;
        ok = mbar_wait(bar_mma, ph_mma, abort_flag, WAIT_CYCLES) && ok;
        ph_mma ^= 1;
        tc_fence_after();
#pragma unroll
        for (int sl = 0; sl < 2; ++sl) {
            const int s0 = 64 * hf + 32 * sl;
            if (s0 >= Nc) continue;  // same decision in the whole warp (hf, Nc uniform)
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
                        float p0 = 0.f, p1 = 0.f, d0 = 0.f, d1 = 0.f;
                        if (km & (1u << j)) {
                            p0 = exp2f(fmaf(__uint_as_float(rs[j]), a.scale_log2, -lse2));
                            d0 = p0 * (__uint_as_float(rd[j]) - dl);
                        }
                        if (km & (2u << j)) {
                            p1 = exp2f(fmaf(__uint_as_float(rs[j + 1]), a.scale_log2, -lse2));
                            d1 = p1 * (__uint_as_float(rd[j + 1]) - dl);
                        }
                        pp[j >> 1] = pack_bf16(p0, p1);
                        pd[j >> 1] = pack_bf16(d0, d1);
                    }
                }
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t off = hf * SUB + swz(rl, sl * 4 + c);
                *reinterpret_cast<uint4 *>(sP + off) = make_uint4(pp[4 * c], pp[4 * c + 1], pp[4 * c + 2], pp[4 * c + 3]);
                *reinterpret_cast<uint4 *>(sDS + off) = make_uint4(pd[4 * c], pd[4 * c + 1], pd[4 * c + 2], pd[4 * c + 3]);
            }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();
        if (tid == 0 && !*abort_flag) {
            tc_fence_after();
            const uint32_t idesc_kv = idesc_bf16(D, true, true);   // A = P^T / dS^T, B = dO / Q (both MN-major)
            const uint32_t idesc_q = idesc_bf16(D, false, true);   // A = dS (K-major), B = K (MN-major)
            if (want_dkdv) {
                for (int kk = 0; kk < Kr / 16; ++kk) {
                    const uint64_t ap = smem_desc(smem_u32(sP) + kk * 2048, SUB, 1024);
                    const uint64_t bdo = smem_desc(smem_u32(sDO) + kk * 2048, SUB, 1024);
                    mma_ss(tmem + TM_DV, ap, bdo, idesc_kv, acc_kv || kk > 0);
                }
                for (int kk = 0; kk < Kr / 16; ++kk) {
                    const uint64_t ads = smem_desc(smem_u32(sDS) + kk * 2048, SUB, 1024);
                    const uint64_t bq = smem_desc(smem_u32(sQ) + kk * 2048, SUB, 1024);
                    mma_ss(tmem + TM_DK, ads, bq, idesc_kv, acc_kv || kk > 0);
                }
            }
            if (want_dq) {
                for (int kk = 0; kk < Nc / 16; ++kk) {
                    const uint64_t ads = smem_desc(smem_u32(sDS) + (kk / 4) * SUB + (kk % 4) * 32, 0, 1024);
                    const uint64_t bk = smem_desc(smem_u32(sK) + kk * 2048, SUB, 1024);
                    mma_ss(tmem + TM_DQ, ads, bk, idesc_q, acc_q || kk > 0);
                }
            }
            mma_commit(bar_mma);
        }
        ok = mbar_wait(bar_mma, ph_mma, abort_flag, WAIT_CYCLES) && ok;
        ph_mma ^= 1;
        tc_fence_after();
    };

    auto load = [&](bool q_side, int row0_q, bool k_side, int row0_k) {
        if constexpr (GATHER) {
            const int end_q = a.gather_end_q ? a.gather_end_q : a.n, end_k = a.gather_end_k ? a.gather_end_k : a.n;
            const bool need_delta = a.delta == nullptr;
            if (q_side && k_side && row0_q == row0_k && end_q == end_k) {
                uint8_t *const d4[4] = {sQ, sDO, sK, sV};
                const void *const s4[4] = {a.q, a.d_o, a.k, a.v};
                if (need_delta) gather_tiles_delta<D, 256, 4, 1>(d4, s4, a.o, s_delta, a.tok, row0_q, end_q, H, h, tid);
                else gather_tiles<D, 256, 4>(d4, s4, a.tok, row0_q, end_q, H, h, tid);
            } else {
                if (q_side) {
                    uint8_t *const d2[2] = {sQ, sDO};
                    const void *const s2[2] = {a.q, a.d_o};
                    if (need_delta) gather_tiles_delta<D, 256, 2, 1>(d2, s2, a.o, s_delta, a.tok, row0_q, end_q, H, h, tid);
                    else gather_tiles<D, 256, 2>(d2, s2, a.tok, row0_q, end_q, H, h, tid);
                }
                if (k_side) {
                    uint8_t *const d2[2] = {sK, sV};
                    const void *const s2[2] = {a.k, a.v};
                    gather_tiles<D, 256, 2>(d2, s2, a.tok, row0_k, end_k, H, h, tid);
                }
            }
            fence_proxy_async_smem();     // generic-proxy writes, read by the MMAs
            __syncthreads();
            return;
        }
        if (tid == 0 && !*abort_flag) {
            mbar_expect_tx(bar_tma, (uint32_t)((q_side ? 2 * NSUB : 0) + (k_side ? 2 * NSUB : 0)) * SUB);
            for (int s = 0; s < NSUB; ++s) {
                if (q_side) {
                    tma_load_3d(sQ + s * SUB, &tm_q, 64 * s, h, row0_q, bar_tma);
                    tma_load_3d(sDO + s * SUB, &tm_do, 64 * s, h, row0_q, bar_tma);
                }
                if (k_side) {
                    tma_load_3d(sK + s * SUB, &tm_k, 64 * s, h, row0_k, bar_tma);
                    tma_load_3d(sV + s * SUB, &tm_v, 64 * s, h, row0_k, bar_tma);
                }
            }
        }
        ok = mbar_wait(bar_tma, ph_tma, abort_flag, WAIT_CYCLES) && ok;
        ph_tma ^= 1;
    };

    // Read an accumulator (this thread's row, its half of the D columns), scale, stage as bf16 into
    // `dst` (NSUB swizzled sub-tiles); rows that live on in the next stage also leave the fp32
    // values in that stage's buffer (`part`), which completes and overwrites them.
    auto drain = [&](uint32_t tm_col, bool have, float scale, float *part, uint8_t *dst) {
#pragma unroll
        for (int sl = 0; sl < D / 64; ++sl) {
            const int c0 = hf * (D / 2) + 32 * sl;
            uint32_t r[32];
            if (have) {
                tmem_ld32(tmem + tm_col + lane_base + c0, r);
                tmem_wait_ld();
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = 0u;
            }
            uint32_t pk[16];
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
                const float x0 = __uint_as_float(r[j]) * scale, x1 = __uint_as_float(r[j + 1]) * scale;
                const float x2 = __uint_as_float(r[j + 2]) * scale, x3 = __uint_as_float(r[j + 3]) * scale;
                if (part != nullptr) *reinterpret_cast<float4 *>(part + c0 + j) = make_float4(x0, x1, x2, x3);
                pk[j >> 1] = pack_bf16(x0, x1);
                pk[(j >> 1) + 1] = pack_bf16(x2, x3);
            }
            uint8_t *d = dst + (c0 >> 6) * SUB;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                *reinterpret_cast<uint4 *>(d + swz(rl, ((c0 & 63) >> 3) + c)) =
                    make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
        }
    };
    // final_merge (gathering kernel, stage 1 after stage 0): the accumulator plus stage 0's partial
    // (`base`) plus stage 2's own gradient (`next`, may be nullptr) go straight to the token's row.
    auto drain_final = [&](uint32_t tm_col, bool have, float scale, const float *base, const float *next,
                           __nv_bfloat16 *out) {
#pragma unroll
        for (int sl = 0; sl < D / 64; ++sl) {
            const int c0 = hf * (D / 2) + 32 * sl;
            uint32_t r[32];
            if (have) {
                tmem_ld32(tmem + tm_col + lane_base + c0, r);
                tmem_wait_ld();
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = 0u;
            }
            if (out == nullptr) continue;
            float x[32];
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
                const float4 y = base != nullptr ? *reinterpret_cast<const float4 *>(base + c0 + j) : make_float4(0.f, 0.f, 0.f, 0.f);
                x[j] = fmaf(__uint_as_float(r[j]), scale, y.x);
                x[j + 1] = fmaf(__uint_as_float(r[j + 1]), scale, y.y);
                x[j + 2] = fmaf(__uint_as_float(r[j + 2]), scale, y.z);
                x[j + 3] = fmaf(__uint_as_float(r[j + 3]), scale, y.w);
            }
            if (next != nullptr) {
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    const float4 y = *reinterpret_cast<const float4 *>(next + c0 + j);
                    x[j] += y.x; x[j + 1] += y.y; x[j + 2] += y.z; x[j + 3] += y.w;
                }
            }
#pragma unroll
            for (int c = 0; c < 4; ++c)
                *reinterpret_cast<uint4 *>(out + c0 + 8 * c) =
                    make_uint4(pack_bf16(x[8 * c], x[8 * c + 1]), pack_bf16(x[8 * c + 2], x[8 * c + 3]),
                               pack_bf16(x[8 * c + 4], x[8 * c + 5]), pack_bf16(x[8 * c + 6], x[8 * c + 7]));
        }
    };
    auto copy_out = [&](const uint8_t *src, void *dst_g) {
        __nv_bfloat16 *g = reinterpret_cast<__nv_bfloat16 *>(dst_g);
        for (int idx = tid; idx < NSUB * 128 * 8; idx += 256) {
            const int t = idx >> 10, rem = idx & 1023, r = rem >> 3, c = rem & 7;
            if (r < nrows) {
                const uint4 v = *reinterpret_cast<const uint4 *>(src + t * SUB + swz(r, c));
                *reinterpret_cast<uint4 *>(g + ((size_t)(r0 + r) * H + h) * D + t * 64 + c * 8) = v;
            }
        }
    };

    const bool run = !empty && !dead;
    const int row = r0 + rl;
    const bool inb = row < r1;
    float *cq = nullptr, *ck = nullptr, *cv = nullptr;
    if constexpr (GATHER) {
        if (inb && !a.final_merge) {      // the drains write the own gradients here; the staged bf16 copies are not used
            if (a.phases != 2) cq = a.own_dq + ((size_t)row * H + h) * D;
            if (a.phases != 1) {
                ck = a.own_dk + ((size_t)row * H + h) * D;
                cv = a.own_dv + ((size_t)row * H + h) * D;
            }
        }
    } else if (inb && a.part_dq != nullptr) {
        const int u = a.up[row];
        if (u >= 0) {
            cq = a.part_dq + ((size_t)u * H + h) * D;
            ck = a.part_dk + ((size_t)u * H + h) * D;
            cv = a.part_dv + ((size_t)u * H + h) * D;
        }
    }

    // final_merge: where this row's three gradients go and what is added to them
    const bool fin = GATHER && a.final_merge;
    const float *fb[3] = {nullptr, nullptr, nullptr}, *fn[3] = {nullptr, nullptr, nullptr};
    __nv_bfloat16 *fo[3] = {nullptr, nullptr, nullptr};
    if constexpr (GATHER) {
        if (fin && inb) {
            const size_t tk = (size_t)a.tok[row];
            const size_t ob = ((size_t)row * H + h) * D;
            if (a.final_merge == 1) { fb[0] = a.carry_dq + ob; fb[1] = a.carry_dk + ob; fb[2] = a.carry_dv + ob; }
            // (final_merge = 2: nothing to add; a launch that walks one side only writes that side's gradients only)
            if (a.final_merge == 1 || a.phases != 2) fo[0] = reinterpret_cast<__nv_bfloat16 *>(a.dq) + (tk * H + h) * D;
            if (a.final_merge == 1 || a.phases != 1) {
                fo[1] = reinterpret_cast<__nv_bfloat16 *>(a.dk) + (tk * H + h) * D;
                fo[2] = reinterpret_cast<__nv_bfloat16 *>(a.dv) + (tk * H + h) * D;
            }
            if (a.next_own_dq != nullptr) {
                const int e2 = a.up[row];
                if (e2 >= 0) {
                    const size_t on = ((size_t)e2 * H + h) * D;
                    fn[0] = a.next_own_dq + on; fn[1] = a.next_own_dk + on; fn[2] = a.next_own_dv + on;
                }
            }
        }
    }

    if (fused) {
        load(true, r0, true, r0);
        tile_pass(r0, r1, r0, r1, true, true, false, false);
        if (!ok && tid == 0) atomicCAS(a.status, 0, HDT_ERR_TIMEOUT);
        if (fin) {
            drain_final(TM_DQ, true, a.scale, fb[0], fn[0], fo[0]);
            drain_final(TM_DK, true, a.scale, fb[1], fn[1], fo[1]);
            drain_final(TM_DV, true, 1.f, fb[2], fn[2], fo[2]);
        } else {
            drain(TM_DQ, true, a.scale, cq, sP);
            drain(TM_DK, true, a.scale, ck, sDS);
            drain(TM_DV, true, 1.f, cv, sQ);
        }
    } else {
        if (run && (!GATHER || a.phases != 2)) {
            // this block as query rows: dQ over the key span
            load(true, r0, false, 0);
            for (int c0 = ka; c0 < kb; c0 += 128) {
                load(false, 0, true, c0);
                tile_pass(r0, r1, c0, kb, true, false, c0 > ka, false);
            }
        }
        if (fin) drain_final(TM_DQ, run, a.scale, fb[0], fn[0], fo[0]);
        else drain(TM_DQ, run, a.scale, cq, sP);
        // dQ leaves now: the second walk reuses sP and (at D = 128) the dQ columns of TMEM
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        if constexpr (!GATHER) copy_out(sP, a.dq);
        __syncthreads();
        if (run && (!GATHER || a.phases != 1)) {
            // this block as keys: dK, dV over the same span taken as query rows
            load(false, 0, true, r0);
            for (int c0 = ka; c0 < kb; c0 += 128) {
                load(true, c0, false, 0);
                tile_pass(c0, kb, r0, r1, false, true, false, c0 > ka);
            }
            if (!ok && tid == 0) atomicCAS(a.status, 0, HDT_ERR_TIMEOUT);
        }
        if (fin) {
            drain_final(TM_DK, run, a.scale, fb[1], fn[1], fo[1]);
            drain_final(TM_DV, run, 1.f, fb[2], fn[2], fo[2]);
        } else {
            drain(TM_DK, run, a.scale, ck, sDS);
            drain(TM_DV, run, 1.f, cv, sQ);
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (!GATHER) {
        if (fused) copy_out(sP, a.dq);   // same decision in every thread
        copy_out(sDS, a.dk);
        copy_out(sQ, a.dv);
    }
    if (warp == 0) tmem_dealloc(tmem, TM_COLS);
}


// ---------------------------------------------------------------------------------------------
// Looping backward for SELF, non-EMPTY blocks at D = 128 (the persistent kernel below covers
// D = 64): the fused pass of k_bwd_tc (S, dP; P, dS; dV, dK, dQ over the dead S / dP columns), but
// the CTA stays resident (one per SM: 224 KB of shared memory, all of TMEM), walks the items
// blockIdx.x, + gridDim.x, ... of queue_split x heads, and requests the four input tiles of the
// next item as soon as the output MMAs of the current one have finished — the gradients are
// staged in tiles of their own, so the loads fly while the CTA drains, stages and stores.
// ---------------------------------------------------------------------------------------------
// FD (fused delta): a.delta is not read; delta[row] = dO[row] . O[row] is computed here: the 2 D / 16 lanes that
// share a token row fetch 16 bytes each of its O and dO rows at the top of the item (past L1) and reduce them
// while S and dP are computed; the sums reach the row's two threads through shared memory.
template <int D, bool FD = false>
__global__ void __launch_bounds__(256, 1) k_bwd_tc_loop(const __grid_constant__ CUtensorMap tm_q,
                                                        const __grid_constant__ CUtensorMap tm_k,
                                                        const __grid_constant__ CUtensorMap tm_v,
                                                        const __grid_constant__ CUtensorMap tm_do,
                                                        const __grid_constant__ StoreMaps sm_out, const BwdStageArgs a) {
    constexpr int NSUB = D / 64;
    constexpr uint32_t TM_S = 0, TM_DP = 128, TM_DV = 0, TM_DK = 128, TM_DQ = 256, TM_COLS = 512;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = sm, *sDO = sQ + NSUB * SUB, *sK = sDO + NSUB * SUB, *sV = sK + NSUB * SUB;
    uint8_t *sP = sV + NSUB * SUB, *sDS = sP + 2 * SUB;     // P, dS; later staging of dQ, dK
    uint8_t *sStg = sDS + 2 * SUB;                          // staging of dV
    uint64_t *bar_in = (uint64_t *)(sStg + NSUB * SUB);
    uint64_t *bar_a = bar_in + 1, *bar_b = bar_in + 2;      // S and dP (two issuing threads); dV, dK, dQ (three)
    uint32_t *slot = (uint32_t *)(bar_in + 3);
    volatile int *abort_flag = (volatile int *)(slot + 1);
    float *s_delta = (float *)(bar_in + 8);                 // FD: dO . O of the item's 128 rows

    const int tid = threadIdx.x, warp = tid >> 5, rl = tid & 127, hf = tid >> 7;
    const int H = a.H, G = gridDim.x;
    const float LOG2E = 1.4426950408889634f;
    const int n_items = a.n_fused * H;
    constexpr int LPR = D / 8, RPP = 256 / LPR, NPASS = 128 / RPP;      // FD: lanes per row, rows per pass, passes

    if (tid == 0) {
        mbar_init(bar_in, 1);
        mbar_init(bar_a, 2);
        mbar_init(bar_b, 3);
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
    // MMAs are issued by lane 0 of warps 0, 1, 2 side by side (a thread needs about 100 cycles per MMA)
    const bool issuer = ((tid & 31) == 0) && warp < 3;
    const bool store_thread = ((tid & 31) == 0) && warp >= 2;     // six threads: two boxes per gradient tensor

    struct It { int valid, r0, r1, h; };
    auto fetch = [&](int i) {
        It x{0, 0, 0, 0};
        if (i < n_items) {
            const int *rec = a.blocks + 5 * (size_t)a.queue_split[i / H];
            x.valid = 1; x.r0 = rec[0]; x.r1 = rec[1]; x.h = i % H;
        }
        return x;
    };
    auto issue_loads = [&](const It &d) {       // thread 0
        mbar_expect_tx(bar_in, (uint32_t)(4 * NSUB) * SUB);
        for (int s = 0; s < NSUB; ++s) {
            tma_load_3d(sQ + s * SUB, &tm_q, 64 * s, d.h, d.r0, bar_in);
            tma_load_3d(sDO + s * SUB, &tm_do, 64 * s, d.h, d.r0, bar_in);
            tma_load_3d(sK + s * SUB, &tm_k, 64 * s, d.h, d.r0, bar_in);
            tma_load_3d(sV + s * SUB, &tm_v, 64 * s, d.h, d.r0, bar_in);
        }
    };
    struct RowStat { int lo, hi, up; float lse, dl; };
    auto load_stat = [&](const It &d) {
        RowStat r{0, 0, -1, 0.f, 0.f};
        const int row = d.r0 + rl;
        if (d.valid && row < d.r1) {
            r.lo = a.rng[2 * row];
            r.hi = a.rng[2 * row + 1];
            r.lse = a.lse[(size_t)d.h * a.T + row];      // natural log; scaled where it is used
            if constexpr (!FD) r.dl = a.delta[(size_t)d.h * a.T + row];
            if (a.part_dq != nullptr) r.up = a.up[row];
        }
        return r;
    };

    if (!dead && n_items > 0) {
        It d0 = fetch((int)blockIdx.x), d1 = fetch((int)blockIdx.x + G);
        RowStat rc = load_stat(d0);
        if (tid == 0 && d0.valid) issue_loads(d0);
        for (int it = 0; d0.valid && !*abort_flag; ++it) {
            const It d2 = fetch((int)blockIdx.x + (it + 2) * G);      // record two items ahead
            const RowStat rn = load_stat(d1);                          // row statistics one item ahead
            const int r0 = d0.r0, r1 = d0.r1, h = d0.h, nrows = r1 - r0;
            const int Nc = (nrows + 15) & ~15;
            uint4 xo[NPASS], xg[NPASS];      // FD: chunk tid % LPR of rows tid / LPR + RPP k of O and dO
            if constexpr (FD) {
#pragma unroll
                for (int k = 0; k < NPASS; ++k) {
                    const int r = tid / LPR + RPP * k;
                    xo[k] = make_uint4(0u, 0u, 0u, 0u);
                    xg[k] = make_uint4(0u, 0u, 0u, 0u);
                    if (r < nrows) {
                        const size_t off = ((size_t)(r0 + r) * H + h) * D + (tid % LPR) * 8;
                        xo[k] = ld_stream16(reinterpret_cast<const __nv_bfloat16 *>(a.o) + off);
                        xg[k] = ld_stream16(reinterpret_cast<const __nv_bfloat16 *>(a.d_o) + off);
                    }
                }
            }
            // the next item's tiles start their way from HBM to L2 now; the loads into shared memory
            // (requested once this item's output MMAs have released the tiles) then find them there
            if (tid == 0 && d1.valid) {
                for (int s = 0; s < NSUB; ++s) {
                    tma_prefetch_3d(&tm_q, 64 * s, d1.h, d1.r0);
                    tma_prefetch_3d(&tm_do, 64 * s, d1.h, d1.r0);
                    tma_prefetch_3d(&tm_k, 64 * s, d1.h, d1.r0);
                    tma_prefetch_3d(&tm_v, 64 * s, d1.h, d1.r0);
                }
            }
            ok = mbar_wait(bar_in, it & 1, abort_flag, WAIT_CYCLES) && ok;
            if (issuer && warp < 2 && !*abort_flag) {      // warp 0: S = Q K^T, warp 1: dP = dO V^T
                tc_fence_after();
                const uint32_t idesc = idesc_bf16(Nc, false, false);
                const uint32_t sa = smem_u32(warp == 0 ? sQ : sDO), sb = smem_u32(warp == 0 ? sK : sV);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk / 4) * SUB + (kk % 4) * 32;
                    mma_ss(tmem + (warp == 0 ? TM_S : TM_DP), smem_desc(sa + off, 0, 1024), smem_desc(sb + off, 0, 1024), idesc, kk > 0);
                }
                mma_commit(bar_a);
            }
            const bool inq = rl < nrows;
            const float lse2 = rc.lse * LOG2E;
            float dl = rc.dl;
            const int jl = max(rc.lo - r0, 0), jh = min(rc.hi - r0, nrows);
            const bool has = inq && jh > jl;
            if constexpr (FD) {      // dO . O of the rows this thread fetched: products, then a sum over the LPR lanes of a row
#pragma unroll
                for (int k = 0; k < NPASS; ++k) {
                    const uint32_t xs[4] = {xo[k].x, xo[k].y, xo[k].z, xo[k].w}, ys[4] = {xg[k].x, xg[k].y, xg[k].z, xg[k].w};
                    float acc = 0.f;
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        acc = fmaf(__uint_as_float(xs[w] << 16), __uint_as_float(ys[w] << 16), acc);
                        acc = fmaf(__uint_as_float(xs[w] & 0xffff0000u), __uint_as_float(ys[w] & 0xffff0000u), acc);
                    }
#pragma unroll
                    for (int m = 1; m < LPR; m <<= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
                    if (tid % LPR == 0) s_delta[tid / LPR + RPP * k] = acc;
                }
            }
            ok = mbar_wait(bar_a, it & 1, abort_flag, WAIT_CYCLES) && ok;
            // the previous item's staged gradients have left shared memory before P and dS overwrite them
            if (store_thread) bulk_wait_read();
            __syncthreads();
            tc_fence_after();
            if constexpr (FD) dl = s_delta[rl];
#pragma unroll
            for (int sl = 0; sl < 2; ++sl) {
                const int s0 = 64 * hf + 32 * sl;
                if (s0 >= Nc) continue;      // same decision in the whole warp
                const uint32_t km = has ? keep_mask<false>(s0, 32, jl, jh, 0, 0, false, false) : 0u;
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
                            float p0 = 0.f, p1 = 0.f, e0 = 0.f, e1 = 0.f;
                            if (km & (1u << j)) {
                                p0 = exp2f(fmaf(__uint_as_float(rs[j]), a.scale_log2, -lse2));
                                e0 = p0 * (__uint_as_float(rd[j]) - dl);
                            }
                            if (km & (2u << j)) {
                                p1 = exp2f(fmaf(__uint_as_float(rs[j + 1]), a.scale_log2, -lse2));
                                e1 = p1 * (__uint_as_float(rd[j + 1]) - dl);
                            }
                            pp[j >> 1] = pack_bf16(p0, p1);
                            pd[j >> 1] = pack_bf16(e0, e1);
                        }
                    }
                }
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t off = hf * SUB + swz(rl, sl * 4 + c);
                    *reinterpret_cast<uint4 *>(sP + off) = make_uint4(pp[4 * c], pp[4 * c + 1], pp[4 * c + 2], pp[4 * c + 3]);
                    *reinterpret_cast<uint4 *>(sDS + off) = make_uint4(pd[4 * c], pd[4 * c + 1], pd[4 * c + 2], pd[4 * c + 3]);
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            __syncthreads();
            if (issuer && !*abort_flag) {
                tc_fence_after();
                const uint32_t idesc_kv = idesc_bf16(D, true, true);   // A = P^T / dS^T, B = dO / Q (both MN-major)
                const uint32_t idesc_q = idesc_bf16(D, false, true);   // A = dS (K-major), B = K (MN-major)
                if (warp == 0) {
                    for (int kk = 0; kk < Nc / 16; ++kk)
                        mma_ss(tmem + TM_DV, smem_desc(smem_u32(sP) + kk * 2048, SUB, 1024),
                               smem_desc(smem_u32(sDO) + kk * 2048, SUB, 1024), idesc_kv, kk > 0);
                } else if (warp == 1) {
                    for (int kk = 0; kk < Nc / 16; ++kk)
                        mma_ss(tmem + TM_DK, smem_desc(smem_u32(sDS) + kk * 2048, SUB, 1024),
                               smem_desc(smem_u32(sQ) + kk * 2048, SUB, 1024), idesc_kv, kk > 0);
                } else {
                    for (int kk = 0; kk < Nc / 16; ++kk)
                        mma_ss(tmem + TM_DQ, smem_desc(smem_u32(sDS) + (kk / 4) * SUB + (kk % 4) * 32, 0, 1024),
                               smem_desc(smem_u32(sK) + kk * 2048, SUB, 1024), idesc_q, kk > 0);
                }
                mma_commit(bar_b);
            }
            ok = mbar_wait(bar_b, it & 1, abort_flag, WAIT_CYCLES) && ok;
            tc_fence_after();
            // the input tiles are free: the next item's loads fly during the drain and the stores
            if (tid == 0 && d1.valid && !*abort_flag) issue_loads(d1);
            // ---- drain: this thread's row, its half of the D columns of each gradient ----
            {
                const uint32_t cols[3] = {TM_DQ, TM_DK, TM_DV};
                uint8_t *dsts[3] = {sP, sDS, sStg};
                float *parts[3] = {a.part_dq, a.part_dk, a.part_dv};
#pragma unroll
                for (int t = 0; t < 3; ++t) {
                    const float sc = (t == 2) ? 1.f : a.scale;
                    float *part = (inq && rc.up >= 0) ? parts[t] + ((size_t)rc.up * H + h) * D : nullptr;
#pragma unroll
                    for (int sl = 0; sl < D / 64; ++sl) {
                        const int c0 = hf * (D / 2) + 32 * sl;
                        uint32_t r[32];
                        tmem_ld32(tmem + cols[t] + lane_base + c0, r);
                        tmem_wait_ld();
                        uint32_t pk[16];
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            const float x0 = __uint_as_float(r[j]) * sc, x1 = __uint_as_float(r[j + 1]) * sc;
                            if (part != nullptr) *reinterpret_cast<float2 *>(part + c0 + j) = make_float2(x0, x1);
                            pk[j >> 1] = pack_bf16(x0, x1);
                        }
                        uint8_t *d = dsts[t] + (c0 >> 6) * SUB;
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            *reinterpret_cast<uint4 *>(d + swz(rl, ((c0 & 63) >> 3) + c)) =
                                make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                    }
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            __syncthreads();
            // TMA stores: rows [0, nrows) of each staged tile as at most two boxes of b rows, b the largest
            // power of two <= min(nrows, 64): [0, b) and [nrows - b, nrows); where the two overlap the same
            // values are written twice.  They read shared memory until the next item's arithmetic is
            // about to overwrite it.
            if (store_thread && !*abort_flag) {
                const int t = (warp - 2) >> 1, second = (warp - 2) & 1;
                const int bx = max(__clz(nrows) - 25, 0);          // box of 64 >> bx rows: 64 for nrows >= 64
                const int b = 64 >> bx;
                const int off = second ? nrows - b : 0;
                const uint8_t *src = (t == 0) ? sP : (t == 1) ? sDS : sStg;
                if (!second || nrows > b)
                    for (int u = 0; u < NSUB; ++u) tma_store_3d(&sm_out.m[t][bx], 64 * u, h, r0 + off, src + u * SUB + off * 128);
                bulk_commit();
            }
            d0 = d1; d1 = d2; rc = rn;
        }
    }
    if (!ok && tid == 0) atomicCAS(a.status, 0, HDT_ERR_TIMEOUT);
    if (store_thread) bulk_wait_read();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TM_COLS);
}

// Cycle counts per phase of k_bwd_tc_p, accumulated by thread 0 of CTA 0 (diagnostics).
__device__ long long g_bwd_phase_cycles[16];
#define HDT_STAMP(i)                                        \
    do {                                                    \
        if (stamp) {                                        \
            const long long now_ = clock64();               \
            ph_acc[i] += now_ - t_last;                     \
            t_last = now_;                                  \
        }                                                   \
    } while (0)

// ---------------------------------------------------------------------------------------------
// Persistent, software-pipelined backward for blocks that are SELF and not EMPTY at D = 64.
// One CTA of 512 threads per SM walks its share of the (block, head) items (queue_split order,
// longest first, round-robin over CTAs).  Inputs are double-buffered: while item i is computed
// the TMA loads of item i+1 are in flight or done and those of item i+2 start as soon as item i's
// output MMAs have finished.  S/dP of item i+1 are issued together with the output MMAs of item i,
// so they run while the CTA drains dQ/dK/dV of item i.
// Thread t: row t % 128 (TMEM lane), column quarter t / 128.
// ---------------------------------------------------------------------------------------------

// SPLIT = 0: self-contained blocks.  SPLIT = 1: the other blocks, split families in two walks (first
// every block as query rows over its key span for dQ, then as keys over the same span taken as query
// rows for dK, dV; S, dP, P, dS of every tile pair are computed twice; no atomics, deterministic).
// SPLIT = 2: the other blocks in ONE walk: every block is taken as keys only and walks its span as
// query tiles; dK and dV accumulate in TMEM as before, and the tile's dQ contribution dS K (a fresh
// accumulator per tile pair) is drained as fp32 into a swizzled staging tile and added to the
// fp32 buffer a.dq_acc [T, H, 64] by two TMA reduce-add copies (the L2 does the additions; the
// order in which the CTAs reach a row is not fixed, so dQ of those rows is reproducible only up to
// fp32 rounding of the sum).  k_dq_finish then scales and converts the sums.
template <int SPLIT, bool DIRS = false>
__global__ void __launch_bounds__(512, 1) k_bwd_tc_p(const __grid_constant__ CUtensorMap tm_q,
                                                     const __grid_constant__ CUtensorMap tm_k,
                                                     const __grid_constant__ CUtensorMap tm_v,
                                                     const __grid_constant__ CUtensorMap tm_do,
                                                     const __grid_constant__ StoreMaps sm_out,
                                                     const __grid_constant__ CUtensorMap tm_acc, const BwdStageArgs a) {
    constexpr int D = 64;
    constexpr uint32_t TM_S = 0, TM_DP = 128, TM_DQ = 256, TM_DK = 320, TM_DV = 384, TM_COLS = 512;
    constexpr int STG = SUB;              // one staged output tile: [128 x 64] bf16, swizzled like the inputs
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sIn = sm;                    // 2 stages x {Q, dO, K, V}
    uint8_t *sP = sm + 8 * SUB;           // 2 sub-tiles; later staging of dQ (sub-tile 0), dK (sub-tile 1)
    uint8_t *sDS = sP + 2 * SUB;          // 2 sub-tiles; later staging of dV (sub-tile 0)
    constexpr bool onewalk = SPLIT == 2;
    uint8_t *sAcc = sDS + 2 * SUB;        // one walk: a tile's dQ contribution as fp32, two swizzled sub-tiles of [128 x 32]
    uint64_t *bar_tma = (uint64_t *)(sAcc + (onewalk ? 2 * SUB : 0));   // [2]
    uint64_t *bar_a = bar_tma + 2, *bar_b = bar_tma + 3;
    uint32_t *slot = (uint32_t *)(bar_tma + 4);
    volatile int *abort_flag = (volatile int *)(slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, rl = tid & 127, qt = tid >> 7;
    const int H = a.H, G = gridDim.x;
    const float LOG2E = 1.4426950408889634f;

    if (tid == 0) {
        mbar_init(&bar_tma[0], 1);
        mbar_init(&bar_tma[1], 1);
        mbar_init(bar_a, 2);   // S and dP are issued by two threads
        mbar_init(bar_b, 3);   // dV, dK, dQ by three
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
    // MMAs are issued by lane 0 of warps 0, 1, 2 in parallel: a single thread needs about 100 cycles
    // per small MMA (descriptor arithmetic), three chains issued side by side hide that
    // MMAs are issued by one elected lane of warps 0 to 2 inside warp-uniform branches (cheaper than
    // under a branch on the thread index: C5 backward 1.33 -> 1.29 ms; the same change made the d = 128
    // looping kernel and the transposed kernel slower, so they keep lane 0)
    // six store threads in six warps: (tensor, first / second box); the MMA-issuing warps 0..2 are left alone
    const bool store_thread = ((tid & 31) == 0) && warp >= 4 && warp < 10;

    // ---- work stream of this CTA ----------------------------------------------------------------
    // A unit is a (block, head); this CTA takes units blockIdx.x, + gridDim.x, ... of its group of
    // queue_split (mode 0: the first n_fused blocks, SELF and not EMPTY; mode 1: the others).
    // A SELF block is one item (both tiles = the block, all three gradients).  A block of a split
    // family is 2 x chunks items: first as query rows over its key span (dQ accumulates in TMEM),
    // then as keys over the same span taken as query rows (dK, dV accumulate).  EMPTY blocks are
    // written as zeros on the spot.  Block ids are fetched two units ahead, records one unit ahead,
    // items two ahead and row statistics one ahead: no global-memory latency between two items.
    constexpr bool split = SPLIT != 0;
    const int unit_base = split ? a.n_fused : 0;
    const int n_units = (split ? (a.nb - a.n_fused) : a.n_fused) * H;
    struct UB { int blk, h; };
    struct Unit { int valid, r0, r1, ka, kb, h, empty; };
    struct Item { int valid, q0, qe, k0, ke, h, r0, nrows, flags, up; };
    constexpr int F_DQ = 1, F_DKDV = 2, F_ACC = 4, F_LAST = 8;
    int unit_next = (int)blockIdx.x;
    auto fetch_ub = [&]() {
        UB x{-1, 0};
        const int u = unit_next;
        unit_next += G;
        if (u < n_units) { x.blk = a.queue_split[unit_base + u / H]; x.h = u % H; }
        return x;
    };
    auto fetch_unit = [&](const UB &x) {
        Unit v{0, 0, 0, 0, 0, x.h, 1};
        if (x.blk >= 0) {
            const int *rec = a.blocks + 5 * (size_t)x.blk;
            v.valid = 1; v.r0 = rec[0]; v.r1 = rec[1]; v.ka = rec[2]; v.kb = rec[3];
            v.empty = (rec[4] & HDT_BLK_EMPTY) ? 1 : 0;
        }
        return v;
    };
    auto block_up = [&](const Unit &v) {   // next-stage index of this thread's row of the block
        return (v.valid && a.part_dq != nullptr && v.r0 + rl < v.r1) ? a.up[v.r0 + rl] : -1;
    };
    UB nn = fetch_ub();
    Unit cur = fetch_unit(nn);
    nn = fetch_ub();
    Unit nxt = fetch_unit(nn);
    nn = fetch_ub();
    int up_cur = block_up(cur);
    int role = 0, chunk = 0;
    auto write_empty = [&](const Unit &v, int up) {   // zero gradients of an EMPTY block, this thread's share
        if (v.r0 + rl < v.r1) {
            const uint4 z = make_uint4(0u, 0u, 0u, 0u);
            const size_t e = ((size_t)(v.r0 + rl) * H + v.h) * D + 16 * qt;
            __nv_bfloat16 *g[3] = {(__nv_bfloat16 *)a.dq, (__nv_bfloat16 *)a.dk, (__nv_bfloat16 *)a.dv};
            float *pt[3] = {a.part_dq, a.part_dk, a.part_dv};
#pragma unroll
            for (int t = 0; t < 3; ++t) {
                *reinterpret_cast<uint4 *>(g[t] + e) = z;
                *reinterpret_cast<uint4 *>(g[t] + e + 8) = z;
                if (up >= 0) {
                    float4 *c4 = reinterpret_cast<float4 *>(pt[t] + ((size_t)up * H + v.h) * D + 16 * qt);
#pragma unroll
                    for (int j = 0; j < 4; ++j) c4[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        }
    };
    auto next_item = [&]() {
        Item x{0, 0, 0, 0, 0, 0, 0, 0, 0, -1};
        while (cur.valid) {
            if (cur.empty) {
                if (role == 0) write_empty(cur, up_cur);
                role = 2;
            }
            if (role < 2) {
                x.valid = 1; x.h = cur.h; x.r0 = cur.r0; x.nrows = cur.r1 - cur.r0; x.up = up_cur;
                if (!split) {
                    x.q0 = cur.r0; x.qe = cur.r1; x.k0 = cur.r0; x.ke = cur.r1;
                    x.flags = F_DQ | F_DKDV | F_LAST;
                    role = 2;
                } else {
                    const int nch = (cur.kb - cur.ka + 127) >> 7, c0 = cur.ka + 128 * chunk;
                    if constexpr (onewalk) {   // keys = the block, query tile = chunk of its span; all three products
                        x.q0 = c0; x.qe = cur.kb; x.k0 = cur.r0; x.ke = cur.r1;
                        x.flags = F_DQ | F_DKDV | (chunk > 0 ? F_ACC : 0) | (chunk == nch - 1 ? F_LAST : 0);
                        if (++chunk == nch) { chunk = 0; role = 2; }
                        return x;
                    }
                    if (role == 0) { x.q0 = cur.r0; x.qe = cur.r1; x.k0 = c0; x.ke = cur.kb; }
                    else { x.q0 = c0; x.qe = cur.kb; x.k0 = cur.r0; x.ke = cur.r1; }
                    x.flags = (role == 0 ? F_DQ : F_DKDV) | (chunk > 0 ? F_ACC : 0) | (chunk == nch - 1 ? F_LAST : 0);
                    if (++chunk == nch) { chunk = 0; ++role; }
                }
                return x;
            }
            cur = nxt;                 // next unit; its record was fetched one unit ago
            up_cur = block_up(cur);
            nxt = fetch_unit(nn);
            nn = fetch_ub();
            role = 0; chunk = 0;
        }
        return x;
    };
    struct RowStat { int lo, hi; float lse2, dl; };
    auto load_stat = [&](const Item &d) {
        RowStat r{0, 0, 0.f, 0.f};
        const int row = d.q0 + rl;
        if (d.valid && row < d.qe) {
            r.lo = a.rng[2 * row];
            r.hi = a.rng[2 * row + 1];
            r.lse2 = a.lse[(size_t)d.h * a.T + row];   // natural log; scaled where it is used
            r.dl = a.delta[(size_t)d.h * a.T + row];
        }
        return r;
    };
    auto issue_tma = [&](int n, const Item &d) {       // thread 0
        uint8_t *st = sIn + (n & 1) * 4 * SUB;
        uint64_t *bar = &bar_tma[n & 1];
        mbar_expect_tx(bar, 4 * SUB);
        tma_load_3d(st, &tm_q, 0, d.h, d.q0, bar);
        tma_load_3d(st + SUB, &tm_do, 0, d.h, d.q0, bar);
        tma_load_3d(st + 2 * SUB, &tm_k, 0, d.h, d.k0, bar);
        tma_load_3d(st + 3 * SUB, &tm_v, 0, d.h, d.k0, bar);
    };
    auto issue_sdp = [&](int n, int Nc) {   // warps 0 (S) and 1 (dP), lane 0; inputs of item n have landed
        const uint32_t st = smem_u32(sIn + (n & 1) * 4 * SUB);
        const uint32_t idesc = idesc_bf16(Nc, false, false);
        const uint32_t a_off = (warp == 0) ? 0u : (uint32_t)SUB, b_off = (warp == 0) ? 2u * SUB : 3u * SUB;
        const uint32_t col = (warp == 0) ? TM_S : TM_DP;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk)
            mma_ss(tmem + col, smem_desc(st + a_off + kk * 32, 0, 1024), smem_desc(st + b_off + kk * 32, 0, 1024), idesc, kk > 0);
        mma_commit(bar_a);
    };
    auto keys16 = [&](const Item &d) { return (min(128, d.ke - d.k0) + 15) & ~15; };

    if (!dead && n_units > 0) {
        Item d0 = next_item(), d1 = next_item(), d2 = next_item();
        RowStat rc = load_stat(d0), rn = rc;
        if (tid == 0 && d0.valid) {
            issue_tma(0, d0);
            if (d1.valid) issue_tma(1, d1);
        }
        if (warp < 2 && d0.valid && elect_one()) {
            ok = mbar_wait(&bar_tma[0], 0, abort_flag, WAIT_CYCLES) && ok;
            if (!*abort_flag) {
                tc_fence_after();
                issue_sdp(0, keys16(d0));
            }
        }
        // one walk: the thread that requests the reduce-add copies of a staged dQ tile, and the tile's place
        const bool red_thread = onewalk && tid == 96;
        int red_q0 = -1, red_h = 0;
        const bool stamp = (tid == 0 && blockIdx.x == 0);
        long long ph_acc[12] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
        long long t_last = clock64();
        int it = 0;
        for (; d0.valid; ++it) {
            HDT_STAMP(9);
            rn = load_stat(d1);   // row statistics of the next item
            const int h = d0.h, k0 = d0.k0;
            const int nq = min(128, d0.qe - d0.q0), nk = min(128, d0.ke - k0);
            const int Nc = (nk + 15) & ~15, Kr = (nq + 15) & ~15;
            const bool inq = d0.q0 + rl < d0.qe;
            const float lse2 = rc.lse2 * LOG2E, dl = rc.dl;
            const int jl = max(rc.lo - k0, 0), jh = min(rc.hi - k0, nk);
            const bool has = inq && jh > jl;
            // direction bits (DIRS instantiations): see dir_ok
            const int e_row = d0.q0 + rl;
            const int c_self = e_row - k0, c_head = (rc.lo < e_row) ? rc.lo - k0 : -0x40000000;
            const bool keep_head = (a.dirs & 1) != 0, keep_rest = (a.dirs & ((rc.lo >= e_row) ? 4 : 2)) != 0;
            const int flags = split ? d0.flags : (F_DQ | F_DKDV | F_LAST);   // constant for self-contained blocks
            uint8_t *st = sIn + (it & 1) * 4 * SUB;

            HDT_STAMP(0);
            // S, dP of this item: warp 0 polls the mbarrier, the other warps sleep at the CTA barrier
            if (warp == 0) ok = mbar_wait(bar_a, it & 1, abort_flag, WAIT_CYCLES) && ok;
            if (store_thread) bulk_wait_read();   // the previous item's staged gradients have left shared memory
            __syncthreads();
            tc_fence_after();
            if constexpr (onewalk) {
                // the previous item's dQ tile is staged (all threads have passed the barrier): add it to the buffer
                if (red_thread && red_q0 >= 0 && !*abort_flag) {
                    tma_reduce_add_3d(&tm_acc, 0, red_h, red_q0, sAcc);
                    tma_reduce_add_3d(&tm_acc, 32, red_h, red_q0, sAcc + SUB);
                    bulk_commit();
                    red_q0 = -1;
                }
            }
            HDT_STAMP(1);
            // ---- P and dS of this thread's 32 columns, in two halves of 16 ----
            if (32 * qt < Nc) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int s0 = 32 * qt + 16 * hh;
                    const uint32_t km = has ? keep_mask<DIRS>(s0, 16, jl, jh, c_self, c_head, keep_head, keep_rest) : 0u;
                    const bool mine = km != 0u;
                    uint32_t pp[8], pd[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) { pp[j] = 0u; pd[j] = 0u; }
                    if (__any_sync(0xffffffffu, mine)) {
                        uint32_t rs[16], rd[16];
                        tmem_ld16(tmem + TM_S + lane_base + s0, rs);
                        tmem_ld16(tmem + TM_DP + lane_base + s0, rd);
                        tmem_wait_ld();
                        if (mine) {
#pragma unroll
                            for (int j = 0; j < 16; j += 2) {
                                float p0 = 0.f, p1 = 0.f, e0 = 0.f, e1 = 0.f;
                                if (km & (1u << j)) {
                                    p0 = exp2f(fmaf(__uint_as_float(rs[j]), a.scale_log2, -lse2));
                                    e0 = p0 * (__uint_as_float(rd[j]) - dl);
                                }
                                if (km & (2u << j)) {
                                    p1 = exp2f(fmaf(__uint_as_float(rs[j + 1]), a.scale_log2, -lse2));
                                    e1 = p1 * (__uint_as_float(rd[j + 1]) - dl);
                                }
                                pp[j >> 1] = pack_bf16(p0, p1);
                                pd[j >> 1] = pack_bf16(e0, e1);
                            }
                        }
                    }
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        const uint32_t off = (qt >> 1) * SUB + swz(rl, (qt & 1) * 4 + hh * 2 + c);
                        *reinterpret_cast<uint4 *>(sP + off) = make_uint4(pp[4 * c], pp[4 * c + 1], pp[4 * c + 2], pp[4 * c + 3]);
                        *reinterpret_cast<uint4 *>(sDS + off) = make_uint4(pd[4 * c], pd[4 * c + 1], pd[4 * c + 2], pd[4 * c + 3]);
                    }
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            HDT_STAMP(2);
            __syncthreads();
            HDT_STAMP(3);
            if (warp < 3 && !*abort_flag && elect_one()) {
                tc_fence_after();
                // descriptors differ only in the start address: add (bytes >> 4) to the low word
                const uint32_t sb = smem_u32(st);
                const uint32_t acc = (flags & F_ACC) ? 1u : 0u;
                if (warp == 0 && (flags & F_DKDV)) {          // dV (+)= P^T dO, contraction over the query rows
                    const uint32_t idesc = idesc_bf16(D, true, true);
                    const uint64_t da = smem_desc(smem_u32(sP), SUB, 1024), db = smem_desc(sb + SUB, SUB, 1024);
                    for (int kk = 0; kk < Kr / 16; ++kk)
                        mma_ss(tmem + TM_DV, da + (uint64_t)(kk * 128), db + (uint64_t)(kk * 128), idesc, acc | (kk > 0));
                } else if (warp == 1 && (flags & F_DKDV)) {   // dK (+)= dS^T Q
                    const uint32_t idesc = idesc_bf16(D, true, true);
                    const uint64_t da = smem_desc(smem_u32(sDS), SUB, 1024), db = smem_desc(sb, SUB, 1024);
                    for (int kk = 0; kk < Kr / 16; ++kk)
                        mma_ss(tmem + TM_DK, da + (uint64_t)(kk * 128), db + (uint64_t)(kk * 128), idesc, acc | (kk > 0));
                } else if (warp == 2 && (flags & F_DQ)) {     // dQ (+)= dS K, contraction over the keys
                    const uint32_t idesc = idesc_bf16(D, false, true);
                    const uint64_t da = smem_desc(smem_u32(sDS), 0, 1024), db = smem_desc(sb + 2 * SUB, SUB, 1024);
                    const uint32_t acc_q = onewalk ? 0u : acc;     // one walk: a fresh dQ contribution per tile pair
                    for (int kk = 0; kk < Nc / 16; ++kk)
                        mma_ss(tmem + TM_DQ, da + (uint64_t)((kk / 4) * (SUB >> 4) + (kk % 4) * 2),
                               db + (uint64_t)(kk * 128), idesc, acc_q | (kk > 0));
                }
                mma_commit(bar_b);   // every issuer arrives, with or without MMAs of its own
                HDT_STAMP(10);
                if (warp < 2 && d1.valid) {   // S, dP of the next item run during this item's drain
                    ok = mbar_wait(&bar_tma[(it + 1) & 1], ((it + 1) >> 1) & 1, abort_flag, WAIT_CYCLES) && ok;
                    HDT_STAMP(11);
                    if (!*abort_flag) {
                        tc_fence_after();
                        issue_sdp(it + 1, keys16(d1));
                    }
                }
            }
            HDT_STAMP(4);
            if (warp == 0) ok = mbar_wait(bar_b, it & 1, abort_flag, WAIT_CYCLES) && ok;   // this item's output MMAs
            if (red_thread) bulk_wait_read();      // the reduce-add copies have read the staging tile
            __syncthreads();
            tc_fence_after();
            HDT_STAMP(5);
            if (tid == 0 && d2.valid && !*abort_flag) issue_tma(it + 2, d2);   // this stage is free again
            if constexpr (onewalk) {
                // this tile pair's dQ contribution: 16 fp32 columns of this thread's query row into the
                // staging tile (sub-tile = column half, 128-byte rows, swizzled); the additions are requested
                // behind the next CTA barrier.  Rows beyond the span's end hold exact zeros (their dS is 0).
                uint32_t r[16];
                tmem_ld16(tmem + TM_DQ + lane_base + 16 * qt, r);
                tmem_wait_ld();
                uint8_t *dst = sAcc + (qt >> 1) * SUB;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    *reinterpret_cast<uint4 *>(dst + swz(rl, (qt & 1) * 4 + j)) = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
                fence_proxy_async_smem();
                red_q0 = d0.q0; red_h = h;
            }
            if (flags & F_LAST) {
                // ---- drain: 16 columns of each finished gradient per thread, staged as bf16 ----
                const int r0 = d0.r0, nrows = d0.nrows;
#pragma unroll
                for (int t = 0; t < 3; ++t) {
                    if (!(flags & (t == 0 ? F_DQ : F_DKDV))) continue;   // same in every thread
                    if (onewalk && t == 0) continue;                     // dQ went to the fp32 buffer tile by tile
                    const uint32_t col = (t == 0) ? TM_DQ : (t == 1) ? TM_DK : TM_DV;
                    const float sc = (t == 2) ? 1.f : a.scale;
                    uint8_t *dst = sP + t * STG;    // staging: one swizzled [128 x 64] tile per tensor
                    uint32_t r[16];
                    tmem_ld16(tmem + col + lane_base + 16 * qt, r);
                    tmem_wait_ld();
                    float x[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) x[j] = __uint_as_float(r[j]) * sc;
                    if (d0.up >= 0) {   // this row lives on in the next stage: its fp32 gradients go there too
                        float *base = (t == 0) ? a.part_dq : (t == 1) ? a.part_dk : a.part_dv;
                        float4 *c4 = reinterpret_cast<float4 *>(base + ((size_t)d0.up * H + h) * D + 16 * qt);
#pragma unroll
                        for (int j = 0; j < 4; ++j) c4[j] = make_float4(x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]);
                    }
                    uint32_t pk[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) pk[j] = pack_bf16(x[2 * j], x[2 * j + 1]);
                    *reinterpret_cast<uint4 *>(dst + swz(rl, 2 * qt)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    *reinterpret_cast<uint4 *>(dst + swz(rl, 2 * qt + 1)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                }
                fence_proxy_async_smem();
                tc_fence_before();
                HDT_STAMP(6);
                __syncthreads();
                HDT_STAMP(7);
                // ---- TMA stores: rows [0, nrows) of each staged tile as at most two boxes of b rows, b the
                // largest power of two <= min(nrows, 64): [0, b) and [nrows - b, nrows).  Where the two
                // overlap the same values are written twice.  (A TMA store request costs its thread and the
                // TMA unit about 100 cycles: the binary decomposition of nrows took up to six per tensor.) ----
                if (store_thread) {
                    const int t = (warp - 4) >> 1, second = (warp - 4) & 1;
                    const int bx = max(__clz(nrows) - 25, 0);          // box of 64 >> bx rows: 64 for nrows >= 64
                    const int b = 64 >> bx;
                    const int off = second ? nrows - b : 0;
                    const bool use = (flags & (t == 0 ? F_DQ : F_DKDV)) && (!second || nrows > b) && !(onewalk && t == 0);
                    if (use) tma_store_3d(&sm_out.m[t][bx], 0, h, r0 + off, sP + t * STG + off * 128);
                    bulk_commit();
                }
            }
            HDT_STAMP(8);
            d0 = d1; d1 = d2; d2 = next_item(); rc = rn;
        }
        if (stamp) {
            for (int i = 0; i < 12; ++i) g_bwd_phase_cycles[i] += ph_acc[i];
            g_bwd_phase_cycles[12] += it;
        }
        if constexpr (onewalk) {       // the last item's dQ tile
            __syncthreads();
            if (red_thread && red_q0 >= 0 && !*abort_flag) {
                tma_reduce_add_3d(&tm_acc, 0, red_h, red_q0, sAcc);
                tma_reduce_add_3d(&tm_acc, 32, red_h, red_q0, sAcc + SUB);
                bulk_commit();
            }
            if (red_thread) bulk_wait_read();
        }
    }
    if (!ok) atomicCAS(a.status, 0, HDT_ERR_TIMEOUT);
    if (store_thread) bulk_wait_read();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TM_COLS);
}

// After the one-walk kernel: dQ of the rows of every block that is neither self-contained nor EMPTY
// is the sum in a.dq_acc times the softmax scale; it goes to dq as bf16 and, for rows that live on in
// the next stage, as fp32 to that stage's buffer.  One CTA per (block after the first n_fused of
// queue_split, head); thread t: 16-byte pieces t, t + 256, ... of the block's [rows x 64] fp32 tile.
// zero_empty: the rows of EMPTY blocks (no key in this stage: PAD, lone roots) get their zero gradients here too,
// also in the next stage's buffers for rows that live on (else the kernel before this one has written them).
__global__ void __launch_bounds__(256) k_dq_finish(const BwdStageArgs a, int zero_empty) {
    const int *rec = a.blocks + 5 * (size_t)a.queue_split[a.n_fused + blockIdx.x];
    const int r0 = rec[0], nrows = rec[1] - r0, h = blockIdx.y, H = a.H;
    if (rec[4] & HDT_BLK_EMPTY) {
        if (!zero_empty) return;
        const uint4 z = make_uint4(0u, 0u, 0u, 0u);
        __nv_bfloat16 *g[3] = {(__nv_bfloat16 *)a.dq, (__nv_bfloat16 *)a.dk, (__nv_bfloat16 *)a.dv};
        float *pt[3] = {a.part_dq, a.part_dk, a.part_dv};
        for (int i = threadIdx.x; i < nrows * 8; i += 256) {      // 16 bytes of a row and tensor per step
            const int r = i >> 3, c = i & 7;
            const size_t row = (size_t)(r0 + r);
            const int u = a.part_dq != nullptr ? a.up[row] : -1;
#pragma unroll
            for (int t = 0; t < 3; ++t) {
                *reinterpret_cast<uint4 *>(g[t] + (row * H + h) * 64 + 8 * c) = z;
                if (u >= 0) {
                    float4 *c4 = reinterpret_cast<float4 *>(pt[t] + ((size_t)u * H + h) * 64 + 8 * c);
                    c4[0] = make_float4(0.f, 0.f, 0.f, 0.f);
                    c4[1] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        }
        return;
    }
    for (int i = threadIdx.x; i < nrows * 16; i += 256) {
        const int r = i >> 4, c = i & 15;
        const size_t row = (size_t)(r0 + r);
        const float4 x = *reinterpret_cast<const float4 *>(a.dq_acc + (row * H + h) * 64 + 4 * c);
        const float4 y = make_float4(x.x * a.scale, x.y * a.scale, x.z * a.scale, x.w * a.scale);
        *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(a.dq) + (row * H + h) * 64 + 4 * c) =
            make_uint2(pack_bf16(y.x, y.y), pack_bf16(y.z, y.w));
        if (a.part_dq != nullptr) {
            const int u = a.up[row];
            if (u >= 0) *reinterpret_cast<float4 *>(a.part_dq + ((size_t)u * H + h) * 64 + 4 * c) = y;
        }
    }
}

template <int D>
static int launch_bwd_tc_t(const BwdStageArgs &a, cudaStream_t st) {
    CUtensorMap tq, tk, tv, tdo;
    int rc = make_tmap_bf16(&tq, a.q, D, a.H, a.T, 128);
    if (rc) return rc;
    rc = make_tmap_bf16(&tk, a.k, D, a.H, a.T, 128);
    if (rc) return rc;
    rc = make_tmap_bf16(&tv, a.v, D, a.H, a.T, 128);
    if (rc) return rc;
    rc = make_tmap_bf16(&tdo, a.d_o, D, a.H, a.T, 128);
    if (rc) return rc;
    constexpr int smem = (4 * (D / 64) + 4) * SUB + 1024 + 64 + 512;
    static DevOnce attr;
    if (!attr.done()) {
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attr.set();
    }
    BwdStageArgs b = a;
    b.rest_only = 0;
    int n_general = a.nb;
    const bool dirs = a.dirs != 7;   // direction bits: the instantiations that apply them
    StoreMaps outs;                  // the looping and persistent kernels store through TMA
    {
        void *outp[3] = {a.dq, a.dk, a.dv};
        for (int t = 0; t < 3; ++t)
            for (int bx = 0; bx < 7; ++bx) {
                rc = make_tmap_bf16(&outs.m[t][bx], outp[t], D, a.H, a.T, 64 >> bx);
                if (rc) return rc;
            }
    }
    if (D == 64 && a.nb > 0 && (!a.no_persistent || a.no_persistent == 4 || a.no_persistent == 6)) {   // (no_persistent == 5: the looping kernel below instead)
        // the persistent kernel takes everything: first the blocks of split families (longest first),
        // then the self-contained blocks
        constexpr int smem_p = 12 * SUB + 1024 + 64, smem_w = 14 * SUB + 1024 + 64;
        static DevOnce attr_p;
        int n_sm = 0;
        if (const int rc_ = sm_count(&n_sm)) return rc_;
        if (!attr_p.done()) {
            HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc_p<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_p));
            HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc_p<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_p));
            HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc_p<0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_p));
            HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc_p<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_p));
            HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc_p<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_w));
            HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc_p<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_w));
            attr_p.set();
        }
        // split families in one walk when the caller supplied the fp32 dQ buffer (zeroed): dQ tiles are
        // added to it and k_dq_finish scales and converts the sums afterwards
        const bool onewalk = a.dq_acc != nullptr && a.nb > a.n_fused;
        CUtensorMap tacc = tq;       // (a valid map in the parameter slot of the kernels that do not use it)
        if (onewalk) {
            rc = make_tmap_f32_acc(&tacc, a.dq_acc, a.H, a.T, 128);
            if (rc) return rc;
        }
        for (int mode = 1; mode >= 0; --mode) {
            const long long units = (long long)(mode ? a.nb - a.n_fused : a.n_fused) * a.H;
            if (units == 0) continue;
            if (mode == 0 && a.no_persistent != 4) {     // (4: the persistent kernel takes these too)
                rc = launch_bwd_tc_fused64(a, tq, tk, tv, tdo, outs, (onewalk && a.self_stream) ? (cudaStream_t)a.self_stream : st);
                if (rc) return rc;
                continue;
            }
            BwdStageArgs c = a;
            c.rest_only = mode;
            const int grid_p = (int)(units < n_sm ? units : n_sm);
            if (g_bwd_walk == 86 || g_bwd_walk == 85) c.phases = g_bwd_walk;                // (clock marks: hdt_debug_bwd_w_marks)
            if (mode && onewalk && (g_bwd_walk == 0 || g_bwd_walk == 86 || g_bwd_walk == 85)) {
                // the warp-specialised one-walk kernel (hdt_attn_tc_bwd_w.cu), then the sums become dQ rows
                rc = launch_bwd_tc_onewalk64(c, tq, tk, tv, tdo, outs, tacc, a.n_empty, st);
                if (rc) return rc;
                BwdStageArgs f = c;
                f.scale = 1.f;      // (this kernel's sums carry softmax_scale already: it is in dS)
                k_dq_finish<<<dim3(a.nb - a.n_fused, a.H), 256, 0, st>>>(f, 1);      // (and the EMPTY blocks' zero rows)
            } else if (mode && onewalk) {
                if (dirs) k_bwd_tc_p<2, true><<<grid_p, 512, smem_w, st>>>(tq, tk, tv, tdo, outs, tacc, c);
                else k_bwd_tc_p<2><<<grid_p, 512, smem_w, st>>>(tq, tk, tv, tdo, outs, tacc, c);
                count_launch();
                HDT_CUDA_CHECK(cudaGetLastError());
                const int n_rest = a.nb - a.n_fused;
                k_dq_finish<<<dim3(n_rest, a.H), 256, 0, st>>>(c, 0);
            } else if (dirs) {
                if (mode) k_bwd_tc_p<1, true><<<grid_p, 512, smem_p, st>>>(tq, tk, tv, tdo, outs, tacc, c);
                else k_bwd_tc_p<0, true><<<grid_p, 512, smem_p, st>>>(tq, tk, tv, tdo, outs, tacc, c);
            } else if (mode) k_bwd_tc_p<1><<<grid_p, 512, smem_p, st>>>(tq, tk, tv, tdo, outs, tacc, c);
            else k_bwd_tc_p<0><<<grid_p, 512, smem_p, st>>>(tq, tk, tv, tdo, outs, tacc, c);
            count_launch();
            HDT_CUDA_CHECK(cudaGetLastError());
        }
        n_general = 0;
    }
    if (((D == 128 && !a.no_persistent) || (D == 64 && a.no_persistent == 5)) && a.n_fused > 0 && !dirs) {
        // self-contained blocks through the looping kernel, the rest through the general one
        constexpr int smem_l = (4 * (D / 64) + 4 + (D / 64)) * SUB + 1024 + 64 + 512;
        static DevOnce attr_l;
        int n_sm_l = 0;
        if (const int rc_ = sm_count(&n_sm_l)) return rc_;
        if (!attr_l.done()) {
            HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc_loop<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_l));
            HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc_loop<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_l));
            attr_l.set();
        }
        const long long items = (long long)a.n_fused * a.H;
        if (a.delta == nullptr) {      // no delta pass ran: the kernel computes dO . O of its rows itself
            if (a.o == nullptr) return set_error(HDT_ERR_INVALID_ARG, "launch_bwd_tc: the fused-delta kernel needs o");
            k_bwd_tc_loop<D, true><<<(int)(items < n_sm_l ? items : n_sm_l), 256, smem_l, st>>>(tq, tk, tv, tdo, outs, a);
        } else k_bwd_tc_loop<D><<<(int)(items < n_sm_l ? items : n_sm_l), 256, smem_l, st>>>(tq, tk, tv, tdo, outs, a);
        count_launch();
        HDT_CUDA_CHECK(cudaGetLastError());
        b.rest_only = 1;
        n_general = a.nb - a.n_fused;
    }
    if (n_general > 0) {
        dim3 grid(n_general, a.H);
        if (dirs) {
            static DevOnce attr_d;
            if (!attr_d.done()) {
                HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc<D, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
                attr_d.set();
            }
            k_bwd_tc<D, false, true><<<grid, 256, smem, st>>>(tq, tk, tv, tdo, b);
        } else k_bwd_tc<D><<<grid, 256, smem, st>>>(tq, tk, tv, tdo, b);
        count_launch();
        HDT_CUDA_CHECK(cudaGetLastError());
    }
    return HDT_OK;
}

// Diagnostics: cycles CTA 0 of the persistent backward spent per phase since the last call
// (12 phases, then the item count); resets the counters.
int read_bwd_phase_cycles(long long *out16) {
    HDT_CUDA_CHECK(cudaMemcpyFromSymbol(out16, g_bwd_phase_cycles, sizeof(long long) * 16));
    long long zero[16] = {0};
    HDT_CUDA_CHECK(cudaMemcpyToSymbol(g_bwd_phase_cycles, zero, sizeof(zero)));
    return HDT_OK;
}

// A stage above 0 in own-gradient mode (a.tok and a.own_* set): one CTA per (block, head).
template <int D>
static int launch_bwd_tc_upper_t(const BwdStageArgs &a, cudaStream_t st) {
    CUtensorMap tq;     // the gathering kernel takes no tensor map; the parameter slots get a valid one
    int rc = make_tmap_bf16(&tq, a.q, D, a.H, a.T, 128);
    if (rc) return rc;
    constexpr int smem = (4 * (D / 64) + 4) * SUB + 1024 + 64 + 512;
    static DevOnce attr;
    if (!attr.done()) {
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_bwd_tc<D, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attr.set();
    }
    BwdStageArgs b = a;
    b.rest_only = 0;
    if (a.dirs != 7) k_bwd_tc<D, true, true><<<dim3(a.nb, a.H), 256, smem, st>>>(tq, tq, tq, tq, b);      // direction bits
    else k_bwd_tc<D, true><<<dim3(a.nb, a.H), 256, smem, st>>>(tq, tq, tq, tq, b);
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;
}

int launch_bwd_tc_upper(const BwdStageArgs &a, int D, cudaStream_t st) {
    if (a.nb == 0) return HDT_OK;
    if (a.tok == nullptr || (!a.final_merge && (a.own_dq == nullptr || a.own_dk == nullptr || a.own_dv == nullptr)) ||
        (a.final_merge == 1 && (a.carry_dq == nullptr || a.carry_dk == nullptr || a.carry_dv == nullptr)) ||
        (a.final_merge == 2 && (a.next_own_dq != nullptr || a.dq == nullptr || a.dk == nullptr || a.dv == nullptr)))
        return set_error(HDT_ERR_INVALID_ARG, "launch_bwd_tc_upper: needs a tok map and own-gradient (or carry) buffers");
    if (D == 64) return launch_bwd_tc_upper_t<64>(a, st);
    if (D == 128) return launch_bwd_tc_upper_t<128>(a, st);
    return set_error(HDT_ERR_UNSUPPORTED, "head_dim %d not supported (64 or 128)", D);
}

int launch_bwd_tc(const BwdStageArgs &a, int D, cudaStream_t st) {
    if (a.nb == 0) return HDT_OK;
    if (D == 64) return launch_bwd_tc_t<64>(a, st);
    if (D == 128) return launch_bwd_tc_t<128>(a, st);
    return set_error(HDT_ERR_UNSUPPORTED, "head_dim %d not supported (64 or 128)", D);
}

}  // namespace hdt
