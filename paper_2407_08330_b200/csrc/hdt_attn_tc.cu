// Tensor-core attention kernels for stage 0 (all tokens, in place) in bf16: TMA-staged tiles,
// tcgen05.mma with accumulators in TMEM, in-tile masking from each row's family range.
//
// Forward, one CTA (128 threads, one thread per query row = one TMEM lane) per (row block, head):
//   TMA   Q[r0..r0+128), K/V[c0..c0+128)  ->  128-byte-swizzled shared memory
//   MMA   S = Q K^T                       ->  TMEM columns [0, 128)
//   rows  tcgen05.ld S, mask columns outside [lo, hi), online softmax, P (bf16) -> shared memory
//   MMA   O (+)= P V                      ->  TMEM columns [128, 128 + D)
//   rows  tcgen05.ld O, 1/l, store O and LSE; rows that also belong to the next stage leave their
//         fp32 partial (O, LSE) in its buffer, and that stage writes their final result
// Blocks are packed from whole families, so nearly every block has a single key chunk equal to
// its own rows (Q, K, V are the same 128 token rows); long families loop over key chunks with
// the running maximum and a rescale of O in TMEM.  Two CTAs fit on an SM at D = 64 (80 KB of
// shared memory, 256 TMEM columns each), which overlaps one CTA's softmax with the other's
// loads and MMAs.
#include <cuda_bf16.h>

#include "hdt_internal.cuh"
#include "hdt_sm100.cuh"
#include "hdt_tmap.cuh"

namespace hdt {
using namespace sm100;

static constexpr int SUB = 16384;                 // bytes of one [128 x 64] bf16 sub-tile
static constexpr long long WAIT_CYCLES = 400000000LL;  // ~0.2 s: bound of every barrier wait

// byte offset of 16-byte chunk c (0..7) of row r inside a swizzled sub-tile
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

// GATHER = true (with SINGLE = false): a stage above 0 computed beside stage 0.  Rows are gathered
// through the stage's tok map by the threads instead of TMA, and the kernel leaves only the
// stage's own partial result per element (fp32 O, LSE, indexed by element) for the chain merge.
// DIRS = true: the index carries direction bits other than 7; entries of the row range that the
// bits switch off are masked as well (dir_ok).
template <int D, bool SINGLE, bool GATHER = false, bool DIRS = false>
__global__ void __launch_bounds__(128) k_fwd_tc(const __grid_constant__ CUtensorMap tm_q,
                                                const __grid_constant__ CUtensorMap tm_k,
                                                const __grid_constant__ CUtensorMap tm_v, const FwdStageArgs a) {
    constexpr int NSUB = D / 64;
    constexpr uint32_t TM_S = 0, TM_O = SINGLE ? 0 : 128, TM_COLS = SINGLE ? 128 : 256;
    // PIPE: blocks that walk several key chunks with TMA loads keep two K tiles: K of chunk i + 1 is
    // requested before S of chunk i is computed, V of chunk i + 1 as soon as P V of chunk i is done
    constexpr bool PIPE = !SINGLE && !GATHER;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = sm;                       // NSUB sub-tiles; reused to stage O
    uint8_t *sK = sQ + NSUB * SUB;
    uint8_t *sV = sK + NSUB * SUB;
    uint8_t *sP = SINGLE ? sQ : sV + NSUB * SUB;   // 2 sub-tiles (128 keys)
    uint8_t *sK1 = sP + 2 * SUB;            // PIPE only: the second K tile
    uint64_t *bar_tma = (uint64_t *)((SINGLE ? sV + NSUB * SUB : sP + 2 * SUB + (PIPE ? NSUB * SUB : 0)));
    uint64_t *bar_mma = bar_tma + 1;
    uint64_t *bar_k1 = bar_tma + 2, *bar_v = bar_tma + 3;   // PIPE only
    uint32_t *slot = (uint32_t *)(bar_tma + 4);
    volatile int *abort_flag = (volatile int *)(slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5;
    // SINGLE: the first n_fused entries of queue_split; rest_only: the blocks after them
    const int blk = SINGLE ? a.queue_split[blockIdx.x]
                           : (a.rest_only ? a.queue_split[a.n_fused + blockIdx.x] : a.queue[blockIdx.x]);
    const int h = blockIdx.y, H = a.H;
    const int *rec = a.blocks + 5 * (size_t)blk;
    const int r0 = rec[0], r1 = rec[1], ka = rec[2], kb = rec[3], fl = rec[4];
    const float NEG = -INFINITY, LN2 = 0.6931471805599453f;

    if (tid == 0) {
        mbar_init(bar_tma, 1);
        mbar_init(bar_mma, 1);
        mbar_init(bar_k1, 1);
        mbar_init(bar_v, 1);
        *abort_flag = (*a.status != 0);     // an earlier failure: do not wait for anything
        fence_mbar_init();
    }
    if (warp == 0) tmem_alloc(slot, TM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *slot;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;

    const int row = r0 + tid;
    const bool inb = row < r1;
    int lo = 0, hi = 0;
    if (inb) { lo = a.rng[2 * row]; hi = a.rng[2 * row + 1]; }
    float m = NEG, l = 0.f;
    uint32_t ph_tma = 0, ph_mma = 0;
    bool ok = true;
    // final_merge (gathering kernel): what the epilogue needs from the other stages is requested now
    float fm_lb = NEG, fm_lu = NEG;
    int fm_tk = 0, fm_e2 = -1;
    if constexpr (GATHER) {
        if (a.final_merge && inb) {
            fm_tk = a.tok[row];
            if (a.carry_lse != nullptr) fm_lb = a.carry_lse[(size_t)row * H + h];
            if (a.next_own_o != nullptr) {
                fm_e2 = a.up[row];
                if (fm_e2 >= 0) fm_lu = a.next_own_lse[(size_t)fm_e2 * H + h];
            }
        }
    }
    const bool empty = (fl & HDT_BLK_EMPTY) != 0;
    const bool dead = (*abort_flag != 0);   // same value in every thread: read after the barrier

    if (!empty && !dead) {
        for (int c0 = ka; c0 < kb; c0 += 128) {
            const int nvalid = min(128, kb - c0);
            const int Nc = (nvalid + 15) & ~15;
            const bool first = (c0 == ka);
            if constexpr (GATHER) {
                if (first && ka == r0 && kb == r1) {     // keys = the block's own rows: one round of loads for all three
                    uint8_t *const d3[3] = {sQ, sK, sV};
                    const void *const s3[3] = {a.q, a.k, a.v};
                    gather_tiles<D, 128, 3>(d3, s3, a.tok, r0, r1, H, h, tid);
                } else {
                    if (first) {
                        uint8_t *const dq_[1] = {sQ};
                        const void *const sq_[1] = {a.q};
                        gather_tiles<D, 128, 1>(dq_, sq_, a.tok, r0, r1, H, h, tid);
                    }
                    uint8_t *const dkv[2] = {sK, sV};
                    const void *const skv[2] = {a.k, a.v};
                    gather_tiles<D, 128, 2>(dkv, skv, a.tok, c0, kb, H, h, tid);
                }
                fence_proxy_async_smem();     // generic-proxy writes, read by the MMA
                __syncthreads();
            } else if constexpr (PIPE) {
                const int ci = (c0 - ka) >> 7;
                if (tid == 0 && !*abort_flag) {   // after a failed wait nothing new is issued
                    if (first) {
                        mbar_expect_tx(bar_tma, (uint32_t)(2 * NSUB) * SUB);
                        mbar_expect_tx(bar_v, (uint32_t)NSUB * SUB);
                        for (int s = 0; s < NSUB; ++s) {
                            tma_load_3d(sQ + s * SUB, &tm_q, 64 * s, h, r0, bar_tma);
                            tma_load_3d(sK + s * SUB, &tm_k, 64 * s, h, c0, bar_tma);
                            tma_load_3d(sV + s * SUB, &tm_v, 64 * s, h, c0, bar_v);
                        }
                    }
                    if (c0 + 128 < kb) {          // K of the next chunk into the tile that S of the previous chunk has left
                        uint64_t *bn = (ci & 1) ? bar_tma : bar_k1;
                        uint8_t *kn = (ci & 1) ? sK : sK1;
                        mbar_expect_tx(bn, (uint32_t)NSUB * SUB);
                        for (int s = 0; s < NSUB; ++s) tma_load_3d(kn + s * SUB, &tm_k, 64 * s, h, c0 + 128, bn);
                    }
                }
                if (!mbar_wait((ci & 1) ? bar_k1 : bar_tma, (ci >> 1) & 1, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) a.status[1] = (1 << 8) | 1; }
            } else {
                if (tid == 0 && !*abort_flag) {   // after a failed wait nothing new is issued
                    mbar_expect_tx(bar_tma, (uint32_t)((first ? NSUB : 0) + 2 * NSUB) * SUB);
                    for (int s = 0; s < NSUB; ++s) {
                        if (first) tma_load_3d(sQ + s * SUB, &tm_q, 64 * s, h, r0, bar_tma);
                        tma_load_3d(sK + s * SUB, &tm_k, 64 * s, h, c0, bar_tma);
                        tma_load_3d(sV + s * SUB, &tm_v, 64 * s, h, c0, bar_tma);
                    }
                }
                if (!mbar_wait(bar_tma, ph_tma, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) a.status[1] = (1 << 8) | 2; }
                ph_tma ^= 1;
            }
            if (tid == 0 && !*abort_flag) {
                tc_fence_after();
                const uint32_t idesc = idesc_bf16(Nc, false, false);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk / 4) * SUB + (kk % 4) * 32;
                    const uint32_t kb_ = smem_u32((PIPE && (((c0 - ka) >> 7) & 1)) ? sK1 : sK);
                    mma_ss(tmem + TM_S, smem_desc(smem_u32(sQ) + off, 0, 1024), smem_desc(kb_ + off, 0, 1024), idesc, kk > 0);
                }
                mma_commit(bar_mma);
            }
            if (!mbar_wait(bar_mma, ph_mma, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) a.status[1] = (1 << 8) | 3; }
            ph_mma ^= 1;
            tc_fence_after();

            // ---- masked online softmax of this row over the chunk's columns ----
            const int jl = max(lo - c0, 0), jh = min(hi - c0, nvalid);
            const bool has = inb && jh > jl;
            const int nsl = (Nc + 31) >> 5;
            // direction bits: column of the row itself, of its parent (none for a head row), and
            // whether the parent entry / every other entry of the range is kept
            const int c_self = row - c0, c_head = (lo < row) ? lo - c0 : -0x40000000;
            const bool keep_head = (a.dirs & 1) != 0, keep_rest = (a.dirs & ((lo >= row) ? 4 : 2)) != 0;
            float mx = NEG;
            for (int k = 0; k < nsl; ++k) {
                const int s0 = 32 * k;
                const uint32_t km = has ? keep_mask<DIRS>(s0, 32, jl, jh, c_self, c_head, keep_head, keep_rest) : 0u;
                const bool mine = km != 0u;
                if (__any_sync(0xffffffffu, mine)) {
                    uint32_t r[32];
                    tmem_ld32(tmem + TM_S + lane_base + s0, r);
                    tmem_wait_ld();
                    if (mine) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (km & (1u << j)) mx = fmaxf(mx, __uint_as_float(r[j]));
                    }
                }
            }
            const float m_new = fmaxf(m, mx * a.scale_log2);
            const float alpha = (m_new == NEG) ? 1.f : exp2f(m - m_new);
            float lsum = 0.f;
            for (int k = 0; k < nsl; ++k) {
                const int s0 = 32 * k;
                const uint32_t km = has ? keep_mask<DIRS>(s0, 32, jl, jh, c_self, c_head, keep_head, keep_rest) : 0u;
                const bool mine = km != 0u;
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[j] = 0u;
                if (__any_sync(0xffffffffu, mine)) {
                    uint32_t r[32];
                    tmem_ld32(tmem + TM_S + lane_base + s0, r);
                    tmem_wait_ld();
                    if (mine) {
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            float p0 = 0.f, p1 = 0.f;
                            if (km & (1u << j)) p0 = exp2f(fmaf(__uint_as_float(r[j]), a.scale_log2, -m_new));
                            if (km & (2u << j)) p1 = exp2f(fmaf(__uint_as_float(r[j + 1]), a.scale_log2, -m_new));
                            // the row sum uses the bf16-rounded probabilities the MMA will see
                            const uint32_t u = pack_bf16(p0, p1);
                            lsum += __uint_as_float(u << 16) + __uint_as_float(u & 0xffff0000u);
                            pk[j >> 1] = u;
                        }
                    }
                }
                uint8_t *dst = sP + (k >> 1) * SUB;
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    *reinterpret_cast<uint4 *>(dst + swz(tid, (k & 1) * 4 + c)) =
                        make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
            }
            // ---- rescale the running O (only after the first chunk) ----
            if (!first && !__all_sync(0xffffffffu, alpha == 1.f)) {
#pragma unroll
                for (int k = 0; k < D / 32; ++k) {
                    uint32_t r[32];
                    tmem_ld32(tmem + TM_O + lane_base + 32 * k, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * alpha);
                    tmem_st32(tmem + TM_O + lane_base + 32 * k, r);
                }
                tmem_wait_st();
            }
            l = l * alpha + lsum;
            m = m_new;
            if constexpr (PIPE) ok = mbar_wait(bar_v, ((c0 - ka) >> 7) & 1, abort_flag, WAIT_CYCLES) && ok;   // V of this chunk
            fence_proxy_async_smem();
            tc_fence_before();
            __syncthreads();
            if (tid == 0 && !*abort_flag) {
                tc_fence_after();
                const uint32_t idesc = idesc_bf16(D, false, true);
                for (int kk = 0; kk < Nc / 16; ++kk) {
                    const uint64_t dp = smem_desc(smem_u32(sP) + (kk / 4) * SUB + (kk % 4) * 32, 0, 1024);
                    const uint64_t dv = smem_desc(smem_u32(sV) + kk * 2048, SUB, 1024);
                    mma_ss(tmem + TM_O, dp, dv, idesc, (!first) || kk > 0);
                }
                mma_commit(bar_mma);
            }
            if (!mbar_wait(bar_mma, ph_mma, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) a.status[1] = (1 << 8) | 4; }
            ph_mma ^= 1;
            tc_fence_after();
            if constexpr (PIPE) {
                if (tid == 0 && c0 + 128 < kb && !*abort_flag) {   // V of the next chunk: the tile is free now
                    mbar_expect_tx(bar_v, (uint32_t)NSUB * SUB);
                    for (int s = 0; s < NSUB; ++s) tma_load_3d(sV + s * SUB, &tm_v, 64 * s, h, c0 + 128, bar_v);
                }
            }
        }
    }
    if (!ok && tid == 0) atomicCAS(a.status, 0, HDT_ERR_TIMEOUT);

    // ---- epilogue: normalise; rows that live on in the next stage also leave their fp32 partial
    // result (O, LSE) there, the next stage completes and overwrites them; stage O, store ----
    float lse = NEG, w0 = 0.f;
    if (l > 0.f) { w0 = 1.f / l; lse = (m + log2f(l)) * LN2; }
    if constexpr (GATHER) {
        if (a.final_merge) {
            // log-sum-exp merge of the three partial results of the element: this stage's (in TMEM,
            // unnormalised), stage 0's, stage 2's; straight to the token's row
            const float lb = fm_lb, lu = fm_lu;
            const float *pb = nullptr, *pu = nullptr;
            const int tk = fm_tk;
            if (inb) {
                if (a.carry_o != nullptr) pb = a.carry_o + ((size_t)row * H + h) * D;
                if (fm_e2 >= 0) pu = a.next_own_o + ((size_t)fm_e2 * H + h) * D;
            }
            const float mx = fmaxf(fmaxf(lse, lb), lu);
            float wo = 0.f, wb = 0.f, wu = 0.f, lse_f = NEG;
            if (mx > NEG) {
                wo = (lse > NEG) ? __expf(lse - mx) : 0.f;
                wb = (lb > NEG) ? __expf(lb - mx) : 0.f;
                wu = (lu > NEG) ? __expf(lu - mx) : 0.f;
                const float tot = wo + wb + wu, inv = 1.f / tot;
                wo *= inv * w0; wb *= inv; wu *= inv;        // (w0 normalises this stage's accumulator)
                lse_f = mx + __logf(tot);
            }
            __nv_bfloat16 *og = reinterpret_cast<__nv_bfloat16 *>(a.o) + ((size_t)tk * H + h) * D;
#pragma unroll
            for (int k = 0; k < D / 32; ++k) {
                uint32_t r[32];
                if (!empty && !dead) {      // uniform in the CTA
                    tmem_ld32(tmem + TM_O + lane_base + 32 * k, r);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = 0u;
                }
                if (inb) {
                    float x[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) x[j] = (wo > 0.f) ? __uint_as_float(r[j]) * wo : 0.f;
                    if (wb > 0.f) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const float4 y = *reinterpret_cast<const float4 *>(pb + 32 * k + j);
                            x[j] = fmaf(wb, y.x, x[j]); x[j + 1] = fmaf(wb, y.y, x[j + 1]);
                            x[j + 2] = fmaf(wb, y.z, x[j + 2]); x[j + 3] = fmaf(wb, y.w, x[j + 3]);
                        }
                    }
                    if (wu > 0.f) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const float4 y = *reinterpret_cast<const float4 *>(pu + 32 * k + j);
                            x[j] = fmaf(wu, y.x, x[j]); x[j + 1] = fmaf(wu, y.y, x[j + 1]);
                            x[j + 2] = fmaf(wu, y.z, x[j + 2]); x[j + 3] = fmaf(wu, y.w, x[j + 3]);
                        }
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        *reinterpret_cast<uint4 *>(og + 32 * k + 8 * c) =
                            make_uint4(pack_bf16(x[8 * c], x[8 * c + 1]), pack_bf16(x[8 * c + 2], x[8 * c + 3]),
                                       pack_bf16(x[8 * c + 4], x[8 * c + 5]), pack_bf16(x[8 * c + 6], x[8 * c + 7]));
                }
            }
            if (inb) a.lse[(size_t)h * a.T + tk] = lse_f;
            tc_fence_before();
            __syncthreads();
            if (warp == 0) tmem_dealloc(tmem, TM_COLS);
            return;
        }
        float *own = inb ? a.own_o + ((size_t)row * H + h) * D : nullptr;
#pragma unroll
        for (int k = 0; k < D / 32; ++k) {
            uint32_t r[32];
            if (!empty && !dead) {      // uniform in the CTA
                tmem_ld32(tmem + TM_O + lane_base + 32 * k, r);
                tmem_wait_ld();
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = 0u;
            }
            if (own != nullptr) {
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    float4 x;
                    x.x = (w0 > 0.f) ? __uint_as_float(r[j]) * w0 : 0.f;
                    x.y = (w0 > 0.f) ? __uint_as_float(r[j + 1]) * w0 : 0.f;
                    x.z = (w0 > 0.f) ? __uint_as_float(r[j + 2]) * w0 : 0.f;
                    x.w = (w0 > 0.f) ? __uint_as_float(r[j + 3]) * w0 : 0.f;
                    *reinterpret_cast<float4 *>(own + 32 * k + j) = x;
                }
            }
        }
        if (inb) a.own_lse[(size_t)row * H + h] = lse;
        tc_fence_before();
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem, TM_COLS);
        return;
    }
    float *po = nullptr;
    if (inb && a.part_o != nullptr) {
        const int u = a.up[row];
        if (u >= 0) {
            po = a.part_o + ((size_t)u * H + h) * D;
            a.part_lse[(size_t)u * H + h] = lse;
        }
    }
#pragma unroll
    for (int k = 0; k < D / 32; ++k) {
        uint32_t r[32];
        if (!empty && !dead) {
            tmem_ld32(tmem + TM_O + lane_base + 32 * k, r);
            tmem_wait_ld();
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] = 0u;
        }
        float x[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) x[j] = (w0 > 0.f) ? __uint_as_float(r[j]) * w0 : 0.f;
        if (po != nullptr) {
#pragma unroll
            for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<float4 *>(po + 32 * k + j) = make_float4(x[j], x[j + 1], x[j + 2], x[j + 3]);
        }
        uint32_t pk[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) pk[j] = pack_bf16(x[2 * j], x[2 * j + 1]);
        uint8_t *dst = sQ + (k >> 1) * SUB;
#pragma unroll
        for (int c = 0; c < 4; ++c)
            *reinterpret_cast<uint4 *>(dst + swz(tid, (k & 1) * 4 + c)) =
                make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
    }
    if (inb) a.lse[(size_t)h * a.T + row] = lse;
    tc_fence_before();
    __syncthreads();
    {
        __nv_bfloat16 *og = reinterpret_cast<__nv_bfloat16 *>(a.o);
        const int nrows = r1 - r0;
        for (int idx = tid; idx < NSUB * 128 * 8; idx += 128) {
            const int t = idx >> 10, rem = idx & 1023, r = rem >> 3, c = rem & 7;
            if (r < nrows) {
                const uint4 v = *reinterpret_cast<const uint4 *>(sQ + t * SUB + swz(r, c));
                *reinterpret_cast<uint4 *>(og + ((size_t)(r0 + r) * H + h) * D + t * 64 + c * 8) = v;
            }
        }
    }
    if (warp == 0) tmem_dealloc(tmem, TM_COLS);
}


// ---------------------------------------------------------------------------------------------
// Looping forward for SELF, non-EMPTY blocks: the single-chunk layout above (P over Q/K, O over
// S), but each CTA stays resident and walks items blockIdx.x, + gridDim.x, ... (queue_split order
// x heads), with 4 (D = 64) or 2 (D = 128) CTAs per SM.  TMEM and barriers are set up once; Q and
// K of the next item are fetched as soon as P V of the current one has finished (P, which lives
// in the Q/K tiles, is dead then), V of the next item once the staged O has left the V tile.
// ---------------------------------------------------------------------------------------------
// Cycle counts per phase, accumulated by thread 0 of CTA 0 (diagnostics): of the looping kernel's
// instrumented instantiation (STAMP), or of the persistent kernel further down.
__device__ long long g_fwd_phase_cycles[16];
__device__ long long g_fwd_timeline[1024][4];   // STAMP: per CTA: global timer at entry, first tiles in, loop end; SM id
__device__ __forceinline__ long long gtime_f() { long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
#define HDT_LSTAMP(i)                                                              \
    do {                                                                           \
        if constexpr (STAMP) {                                                     \
            if (tid == 0 && blockIdx.x == 0) {                                     \
                const long long now_ = clock64();                                  \
                atomicAdd((unsigned long long *)&g_fwd_phase_cycles[i], (unsigned long long)(now_ - t_last)); \
                t_last = now_;                                                     \
            }                                                                      \
        }                                                                          \
    } while (0)

template <int D, bool DIRS = false, bool STAMP = false>
__global__ void __launch_bounds__(128) k_fwd_tc_loop(const __grid_constant__ CUtensorMap tm_q,
                                                     const __grid_constant__ CUtensorMap tm_k,
                                                     const __grid_constant__ CUtensorMap tm_v,
                                                     const __grid_constant__ OutMaps om, const FwdStageArgs a) {
    constexpr int NSUB = D / 64;
    // S (N <= 128 columns); P (bf16, two per column) is written over its first half as the rows are
    // exponentiated and is the A operand of O = P V; O lies beside it
    constexpr uint32_t TM_O = (D == 64) ? 64 : 128, TM_COLS = (D == 64) ? 128 : 256;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = sm, *sK = sQ + NSUB * SUB, *sV = sK + NSUB * SUB;
    uint64_t *bar_qk = (uint64_t *)(sV + NSUB * SUB);
    uint64_t *bar_v = bar_qk + 1, *bar_mma = bar_qk + 2;
    uint32_t *slot = (uint32_t *)(bar_qk + 3);
    volatile int *abort_flag = (volatile int *)(slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int H = a.H, G = gridDim.x;
    if constexpr (STAMP) { if (tid == 0 && blockIdx.x < 1024) { g_fwd_timeline[blockIdx.x][0] = gtime_f(); unsigned sm_; asm("mov.u32 %0, %%smid;" : "=r"(sm_)); g_fwd_timeline[blockIdx.x][3] = sm_; g_fwd_timeline[blockIdx.x][1] = 0; g_fwd_timeline[blockIdx.x][2] = 0; } }
    // Counts not yet known to the host (the index build is still in flight when this kernel is
    // queued): they are read from the index header, and the partial buffers of stage 1 are laid
    // out from its element count the way the host does it (results, then LSE, 256-byte aligned).
    int n_fused = a.n_fused;
    float *part_o = a.part_o, *part_lse = a.part_lse;
    if (a.hdr != nullptr) {
        const DevHeader *hd = a.hdr;
        n_fused = (hd->status == 0) ? hd->st[0].n_fused : 0;
        const size_t n1 = (size_t)hd->st[1].n;
        const size_t b_o = (sizeof(float) * n1 * H * D + 255) & ~size_t(255), b_l = (sizeof(float) * n1 * H + 255) & ~size_t(255);
        if (n1 == 0) {
            part_o = nullptr;
            part_lse = nullptr;
        } else if (part_o == nullptr || b_o + b_l > a.ws_bytes) {
            n_fused = 0;            // the host finds the same after its wait and reports the workspace error
        } else {
            part_lse = reinterpret_cast<float *>(reinterpret_cast<char *>(part_o) + b_o);
        }
    }
    const int n_items = n_fused * H;
    const float NEG = -INFINITY, LN2 = 0.6931471805599453f;

    struct Desc { int r0, r1, ka, kb, h; };
    auto load_desc = [&](int item) {
        Desc d{0, 0, 0, 0, 0};
        if (item < n_items) {
            const int *rec = a.blocks + 5 * (size_t)a.queue_split[item / H];
            d.r0 = rec[0]; d.r1 = rec[1]; d.ka = rec[2]; d.kb = rec[3]; d.h = item % H;
        }
        return d;
    };
    auto issue_qk = [&](const Desc &d) {   // thread 0
        mbar_expect_tx(bar_qk, (uint32_t)(2 * NSUB) * SUB);
        for (int s = 0; s < NSUB; ++s) {
            tma_load_3d(sQ + s * SUB, &tm_q, 64 * s, d.h, d.r0, bar_qk);
            tma_load_3d(sK + s * SUB, &tm_k, 64 * s, d.h, d.ka, bar_qk);
        }
    };
    auto issue_v = [&](const Desc &d) {    // thread 0
        mbar_expect_tx(bar_v, (uint32_t)NSUB * SUB);
        for (int s = 0; s < NSUB; ++s) tma_load_3d(sV + s * SUB, &tm_v, 64 * s, d.h, d.ka, bar_v);
    };

    if (tid == 0) {
        mbar_init(bar_qk, 1);
        mbar_init(bar_v, 1);
        mbar_init(bar_mma, 1);
        fence_mbar_init();
        // the first item's tiles are requested before anything else is set up
        if ((int)blockIdx.x < n_items) {
            const Desc d = load_desc((int)blockIdx.x);
            issue_qk(d);
            issue_v(d);
        }
        *abort_flag = (*a.status != 0);
    }
    if (warp == 0) tmem_alloc(slot, TM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *slot;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    const bool dead = (*abort_flag != 0);
    bool ok = true;

    if (!dead && (int)blockIdx.x < n_items) {
        Desc dc = load_desc((int)blockIdx.x), dn = load_desc((int)blockIdx.x + G);
        uint32_t ph = 0;           // phase of bar_qk and bar_v (one completion of each per item)
        uint32_t ph_mma = 0;
        long long t_last = STAMP ? clock64() : 0;
        for (int item = (int)blockIdx.x; item < n_items; item += G) {
            const Desc dn2 = load_desc(item + 2 * G);   // needed two iterations from now
            const int r0 = dc.r0, r1 = dc.r1, ka = dc.ka, kb = dc.kb, h = dc.h;
            const bool have_next = item + G < n_items;
            // D = 128 (two CTAs per SM): the next item's tiles start their way from HBM to L2 now; the
            // loads into shared memory (requested once this item has released the tiles) then find
            // them there.  (At D = 64 four CTAs per SM hide that latency already; measured: the
            // prefetch costs 6 % there and gains 12 % here.)
            if (D == 128 && tid == 0 && have_next) {
                for (int s = 0; s < NSUB; ++s) {
                    tma_prefetch_3d(&tm_q, 64 * s, dn.h, dn.r0);
                    tma_prefetch_3d(&tm_k, 64 * s, dn.h, dn.ka);
                    tma_prefetch_3d(&tm_v, 64 * s, dn.h, dn.ka);
                }
            }
            const int row = r0 + tid;
            const bool inb = row < r1;
            int lo = 0, hi = 0, up = -1;
            if (inb) {
                lo = a.rng[2 * row];
                hi = a.rng[2 * row + 1];
                if (part_o != nullptr) up = a.up[row];
            }
            const int nvalid = min(128, kb - ka), Nc = (nvalid + 15) & ~15;

            HDT_LSTAMP(0);
            if (!mbar_wait(bar_qk, ph, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) { a.status[1] = (2 << 8) | 1; a.status[2] = item; } }
            if (tid == 32 && item != (int)blockIdx.x) {      // V of this item, into the tile the previous item's stores read
                bulk_wait_read();
                if (!*abort_flag) issue_v(dc);
            }
            HDT_LSTAMP(1);
            if constexpr (STAMP) { if (tid == 0 && item == (int)blockIdx.x && blockIdx.x < 1024) g_fwd_timeline[blockIdx.x][1] = gtime_f(); }
            if (warp == 0 && !*abort_flag && elect_one()) {
                tc_fence_after();
                const uint32_t idesc = idesc_bf16(Nc, false, false);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk / 4) * SUB + (kk % 4) * 32;
                    mma_ss(tmem, smem_desc(smem_u32(sQ) + off, 0, 1024), smem_desc(smem_u32(sK) + off, 0, 1024), idesc, kk > 0);
                }
                mma_commit(bar_mma);
            }
            if (!mbar_wait(bar_mma, ph_mma, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) { a.status[1] = (2 << 8) | 2; a.status[2] = item; } }
            ph_mma ^= 1;
            tc_fence_after();
            HDT_LSTAMP(2);

            // ---- masked softmax of this row (one chunk: no running maximum needed) ----
            const int jl = max(lo - ka, 0), jh = min(hi - ka, nvalid);
            const bool has = inb && jh > jl;
            const int nsl = (Nc + 31) >> 5;
            // direction bits (DIRS instantiation): see dir_ok
            const int c_self = row - ka, c_head = (lo < row) ? lo - ka : -0x40000000;
            const bool keep_head = (a.dirs & 1) != 0, keep_rest = (a.dirs & ((lo >= row) ? 4 : 2)) != 0;
            float mx = NEG;
            for (int k = 0; k < nsl; ++k) {
                const int s0 = 32 * k;
                const uint32_t km = has ? keep_mask<DIRS>(s0, 32, jl, jh, c_self, c_head, keep_head, keep_rest) : 0u;
                const bool mine = km != 0u;
                if (__any_sync(0xffffffffu, mine)) {
                    uint32_t r[32];
                    tmem_ld32(tmem + lane_base + s0, r);
                    tmem_wait_ld();
                    if (mine) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (km & (1u << j)) mx = fmaxf(mx, __uint_as_float(r[j]));
                    }
                }
            }
            HDT_LSTAMP(3);
            const float m = mx * a.scale_log2;
            float l = 0.f;
            for (int k = 0; k < nsl; ++k) {
                const int s0 = 32 * k;
                const uint32_t km = has ? keep_mask<DIRS>(s0, 32, jl, jh, c_self, c_head, keep_head, keep_rest) : 0u;
                const bool mine = km != 0u;
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[j] = 0u;
                if (__any_sync(0xffffffffu, mine)) {
                    uint32_t r[32];
                    tmem_ld32(tmem + lane_base + s0, r);
                    tmem_wait_ld();
                    if (mine) {
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            float p0 = 0.f, p1 = 0.f;
                            if (km & (1u << j)) p0 = exp2f(fmaf(__uint_as_float(r[j]), a.scale_log2, -m));
                            if (km & (2u << j)) p1 = exp2f(fmaf(__uint_as_float(r[j + 1]), a.scale_log2, -m));
                            const uint32_t u = pack_bf16(p0, p1);   // the row sum uses the rounded values the MMA sees
                            l += __uint_as_float(u << 16) + __uint_as_float(u & 0xffff0000u);
                            pk[j >> 1] = u;
                        }
                    }
                }
                // keys s0..s0+31 are K indices s0..s0+31 of the P V MMA: 16 packed columns, over S columns
                // this thread has already read
                tmem_st16(tmem + lane_base + 16 * k, pk);
            }
            tmem_wait_st();
            tc_fence_before();
            HDT_LSTAMP(4);
            __syncthreads();
            HDT_LSTAMP(5);
            // Q, K of the next item (S has consumed the tiles; only after this barrier has every thread
            // seen the current phase of their barrier, so that re-arming it cannot overtake anybody)
            if (tid == 0 && have_next && !*abort_flag) issue_qk(dn);
            if (!mbar_wait(bar_v, ph, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) { a.status[1] = (2 << 8) | 3; a.status[2] = item; } }
            ph ^= 1;
            if (warp == 0 && !*abort_flag && elect_one()) {
                tc_fence_after();
                const uint32_t idesc = idesc_bf16(D, false, true);
                for (int kk = 0; kk < Nc / 16; ++kk)
                    mma_ts(tmem + TM_O, tmem + 8 * kk, smem_desc(smem_u32(sV) + kk * 2048, SUB, 1024), idesc, kk > 0);
                mma_commit(bar_mma);
            }
            if (!mbar_wait(bar_mma, ph_mma, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) { a.status[1] = (2 << 8) | 4; a.status[2] = item; } }
            ph_mma ^= 1;
            tc_fence_after();
            HDT_LSTAMP(6);
            // ---- drain O, stage it (bf16) in the V tile, store ----
            float lse = NEG, w0 = 0.f;
            if (l > 0.f) { w0 = 1.f / l; lse = (m + log2f(l)) * LN2; }
            float *po = nullptr;
            if (up >= 0) {
                po = part_o + ((size_t)up * H + h) * D;
                part_lse[(size_t)up * H + h] = lse;
            }
#pragma unroll
            for (int k = 0; k < D / 32; ++k) {
                uint32_t r[32];
                tmem_ld32(tmem + TM_O + lane_base + 32 * k, r);
                tmem_wait_ld();
                float x[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) x[j] = (w0 > 0.f) ? __uint_as_float(r[j]) * w0 : 0.f;
                if (po != nullptr) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *reinterpret_cast<float4 *>(po + 32 * k + j) = make_float4(x[j], x[j + 1], x[j + 2], x[j + 3]);
                }
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[j] = pack_bf16(x[2 * j], x[2 * j + 1]);
                uint8_t *dst = sV + (k >> 1) * SUB;
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    *reinterpret_cast<uint4 *>(dst + swz(tid, (k & 1) * 4 + c)) =
                        make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
            }
            if (inb) a.lse[(size_t)h * a.T + row] = lse;
            fence_proxy_async_smem();
            tc_fence_before();
            HDT_LSTAMP(7);
            __syncthreads();
            HDT_LSTAMP(8);
            // The staged rows leave through TMA stores: rows [0, nrows) as at most two boxes of b rows, b
            // the largest power of two <= min(nrows, 64) (where the two overlap the same values are
            // written twice).  One thread of warp 1 requests them; at the top of the next item, once it
            // has seen that item's Q and K arrive, it waits until the stores have read the tile and
            // requests V into it.  (Not here: a thread that lags behind the others by that wait could
            // miss a phase of the Q / K barrier, which thread 0 re-arms as soon as S is there.)
            if (tid == 32 && !*abort_flag) {
                const int nrows = r1 - r0;
                const int bx = max(__clz(nrows) - 25, 0);          // box of 64 >> bx rows: 64 for nrows >= 64
                const int b = 64 >> bx;
                for (int s2 = 0; s2 < NSUB; ++s2) {
                    tma_store_3d(&om.m[bx], 64 * s2, h, r0, sV + s2 * SUB);
                    if (nrows > b) tma_store_3d(&om.m[bx], 64 * s2, h, r0 + nrows - b, sV + s2 * SUB + (nrows - b) * 128);
                }
                bulk_commit();
            }
            HDT_LSTAMP(9);
            HDT_LSTAMP(10);
            if constexpr (STAMP) { if (tid == 0 && blockIdx.x == 0) atomicAdd((unsigned long long *)&g_fwd_phase_cycles[12], 1ull); }
            dc = dn; dn = dn2;
        }
    }
    if (tid == 32) bulk_wait_read();       // the last item's stores have read the tile
    if (dead && (int)blockIdx.x < n_items) {     // an earlier failure: only let the tiles requested above land
        volatile int none = 0;
        (void)mbar_wait(bar_qk, 0, &none, WAIT_CYCLES);
        (void)mbar_wait(bar_v, 0, &none, WAIT_CYCLES);
    }
    if constexpr (STAMP) { if (tid == 0 && blockIdx.x < 1024) g_fwd_timeline[blockIdx.x][2] = gtime_f(); }
    if (!ok && tid == 0) atomicCAS(a.status, 0, HDT_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TM_COLS);
}

// Cycle counts per phase of k_fwd_tc_p, accumulated by thread 0 of CTA 0 (diagnostics).
#ifdef HDT_WORKBENCH      // (the persistent single-CTA-per-SM forward: kept for comparisons, option "no_persistent" = 2)
#define HDT_STAMP(i)                                        \
    do {                                                    \
        if (stamp) {                                        \
            const long long now_ = clock64();               \
            ph_acc[i] += now_ - t_last;                     \
            t_last = now_;                                  \
        }                                                   \
    } while (0)

// ---------------------------------------------------------------------------------------------
// Persistent, software-pipelined forward for blocks that are SELF and not EMPTY at D = 64.
// One CTA of 512 threads per SM walks its share of the (block, head) items in queue_split order.
// Q/K/V of the next two items are in flight or resident (double-buffered TMA); S of item i+1 is
// issued together with O = P V of item i and runs while the CTA drains O.
// Thread t: row t % 128 (TMEM lane), column quarter t / 128; the four threads of a row exchange
// their partial row maximum and row sum through shared memory.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(512, 1) k_fwd_tc_p(const __grid_constant__ CUtensorMap tm_q,
                                                     const __grid_constant__ CUtensorMap tm_k,
                                                     const __grid_constant__ CUtensorMap tm_v, const FwdStageArgs a) {
    constexpr int D = 64;
    constexpr uint32_t TM_S = 0, TM_O = 128, TM_COLS = 256;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sIn = sm;                    // 2 stages x {Q, K, V}
    uint8_t *sP = sm + 6 * SUB;           // 2 sub-tiles; reused to stage O (rows padded to 144 bytes) once P V is done
    float *s_red = (float *)(sP + 2 * SUB);              // [4][128] partial row max, then partial row sums
    uint64_t *bar_tma = (uint64_t *)(s_red + 4 * 128);   // [2]
    uint64_t *bar_s = bar_tma + 2, *bar_o = bar_tma + 3;
    uint32_t *slot = (uint32_t *)(bar_tma + 4);
    volatile int *abort_flag = (volatile int *)(slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, rl = tid & 127, qt = tid >> 7;
    const int H = a.H, G = gridDim.x;
    const int n_items = a.n_fused * H;
    const int my_count = ((int)blockIdx.x < n_items) ? (n_items - (int)blockIdx.x + G - 1) / G : 0;
    const float NEG = -INFINITY, LN2 = 0.6931471805599453f;

    if (tid == 0) {
        mbar_init(&bar_tma[0], 1);
        mbar_init(&bar_tma[1], 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
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

    struct Desc { int r0, r1, h; };
    auto load_blk = [&](int i) { return a.queue_split[((int)blockIdx.x + i * G) / H]; };
    auto load_rec = [&](int i, int blk) {
        Desc d;
        d.h = ((int)blockIdx.x + i * G) % H;
        d.r0 = a.blocks[5 * (size_t)blk];
        d.r1 = a.blocks[5 * (size_t)blk + 1];
        return d;
    };
    struct RowStat { int lo, hi, up; };
    auto load_stat = [&](const Desc &d) {
        RowStat r{0, 0, -1};
        const int row = d.r0 + rl;
        if (row < d.r1) {
            r.lo = a.rng[2 * row];
            r.hi = a.rng[2 * row + 1];
            if (a.part_o != nullptr) r.up = a.up[row];
        }
        return r;
    };
    auto issue_tma = [&](int i, const Desc &d) {       // thread 0
        uint8_t *st = sIn + (i & 1) * 3 * SUB;
        uint64_t *bar = &bar_tma[i & 1];
        mbar_expect_tx(bar, 3 * SUB);
        tma_load_3d(st, &tm_q, 0, d.h, d.r0, bar);
        tma_load_3d(st + SUB, &tm_k, 0, d.h, d.r0, bar);
        tma_load_3d(st + 2 * SUB, &tm_v, 0, d.h, d.r0, bar);
    };
    auto issue_s = [&](int i, int Nc) {   // one thread; inputs of item i have landed
        const uint32_t st = smem_u32(sIn + (i & 1) * 3 * SUB);
        const uint32_t idesc = idesc_bf16(Nc, false, false);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk)
            mma_ss(tmem + TM_S, smem_desc(st + kk * 32, 0, 1024), smem_desc(st + SUB + kk * 32, 0, 1024), idesc, kk > 0);
        mma_commit(bar_s);
    };

    if (!dead && my_count > 0) {
        Desc dc = load_rec(0, load_blk(0)), dn = dc, dn2 = dc;
        if (my_count > 1) dn = load_rec(1, load_blk(1));
        int blk2 = (my_count > 2) ? load_blk(2) : 0;
        RowStat rc = load_stat(dc), rn = rc;
        if (tid == 0) {
            issue_tma(0, dc);
            if (my_count > 1) issue_tma(1, dn);
            ok = mbar_wait(&bar_tma[0], 0, abort_flag, WAIT_CYCLES) && ok;
            if (!*abort_flag) {
                tc_fence_after();
                issue_s(0, (dc.r1 - dc.r0 + 15) & ~15);
            }
        }
        const bool stamp = (tid == 0 && blockIdx.x == 0);
        long long ph_acc[12] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
        long long t_last = clock64();
        for (int it = 0; it < my_count; ++it) {
            HDT_STAMP(9);
            if (it + 2 < my_count) dn2 = load_rec(it + 2, blk2);
            if (it + 3 < my_count) blk2 = load_blk(it + 3);
            if (it + 1 < my_count) rn = load_stat(dn);
            const int r0 = dc.r0, r1 = dc.r1, h = dc.h;
            const int nrows = r1 - r0, Nc = (nrows + 15) & ~15;
            const bool inb = r0 + rl < r1;
            const int jl = max(rc.lo - r0, 0), jh = min(rc.hi - r0, nrows);
            const bool has = inb && jh > jl;
            uint8_t *st = sIn + (it & 1) * 3 * SUB;

            HDT_STAMP(0);
            if (warp == 0) ok = mbar_wait(bar_s, it & 1, abort_flag, WAIT_CYCLES) && ok;   // S of this item
            __syncthreads();   // also: the previous item's staged O has been stored
            tc_fence_after();
            HDT_STAMP(1);
            // ---- this thread's 32 columns of S, kept in registers across both passes ----
            const int s0 = 32 * qt;
            const bool active = s0 < Nc;                       // same in the whole warp
            const bool mine = has && jl < s0 + 32 && jh > s0;
            uint32_t sv[32];
            bool loaded = false;
            float mx = NEG;
            if (active && __any_sync(0xffffffffu, mine)) {
                tmem_ld32(tmem + TM_S + lane_base + s0, sv);
                tmem_wait_ld();
                loaded = true;
                if (mine) {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (s0 + j >= jl && s0 + j < jh) mx = fmaxf(mx, __uint_as_float(sv[j]));
                }
            }
            s_red[qt * 128 + rl] = mx;
            HDT_STAMP(2);
            __syncthreads();
            const float mrow = fmaxf(fmaxf(s_red[rl], s_red[128 + rl]), fmaxf(s_red[256 + rl], s_red[384 + rl])) * a.scale_log2;
            __syncthreads();   // every thread has read the maxima before the sums overwrite them
            HDT_STAMP(3);
            float lsum = 0.f;
            if (active) {
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[j] = 0u;
                if (loaded && mine) {
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        float p0 = 0.f, p1 = 0.f;
                        if (s0 + j >= jl && s0 + j < jh) p0 = exp2f(fmaf(__uint_as_float(sv[j]), a.scale_log2, -mrow));
                        if (s0 + j + 1 >= jl && s0 + j + 1 < jh) p1 = exp2f(fmaf(__uint_as_float(sv[j + 1]), a.scale_log2, -mrow));
                        const uint32_t u = pack_bf16(p0, p1);
                        lsum += __uint_as_float(u << 16) + __uint_as_float(u & 0xffff0000u);
                        pk[j >> 1] = u;
                    }
                }
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    *reinterpret_cast<uint4 *>(sP + (qt >> 1) * SUB + swz(rl, (qt & 1) * 4 + c)) =
                        make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
            }
            s_red[qt * 128 + rl] = lsum;
            fence_proxy_async_smem();
            tc_fence_before();
            HDT_STAMP(4);
            __syncthreads();
            HDT_STAMP(5);
            if ((tid & 31) == 0 && warp < 2 && !*abort_flag) {
                tc_fence_after();
                if (warp == 0) {   // O = P V
                    const uint32_t idesc = idesc_bf16(D, false, true);
                    const uint64_t da = smem_desc(smem_u32(sP), 0, 1024), db = smem_desc(smem_u32(st) + 2 * SUB, SUB, 1024);
                    const int nk = Nc / 16;
                    for (int kk = 0; kk < nk; ++kk)
                        mma_ss(tmem + TM_O, da + (uint64_t)((kk / 4) * (SUB >> 4) + (kk % 4) * 2), db + (uint64_t)(kk * 128),
                               idesc, kk > 0);
                    mma_commit(bar_o);
                } else if (it + 1 < my_count) {   // S of the next item runs during this item's drain
                    ok = mbar_wait(&bar_tma[(it + 1) & 1], ((it + 1) >> 1) & 1, abort_flag, WAIT_CYCLES) && ok;
                    if (!*abort_flag) {
                        tc_fence_after();
                        issue_s(it + 1, (dn.r1 - dn.r0 + 15) & ~15);
                    }
                }
            }
            const float l = s_red[rl] + s_red[128 + rl] + s_red[256 + rl] + s_red[384 + rl];
            HDT_STAMP(6);
            if (warp == 0) ok = mbar_wait(bar_o, it & 1, abort_flag, WAIT_CYCLES) && ok;   // O of this item
            __syncthreads();
            tc_fence_after();
            HDT_STAMP(7);
            if (tid == 0 && it + 2 < my_count && !*abort_flag) issue_tma(it + 2, dn2);   // this stage is free again
            // ---- drain: 16 columns of O per thread ----
            {
                float lse = NEG, w0 = 0.f;
                if (l > 0.f) { w0 = 1.f / l; lse = (mrow + log2f(l)) * LN2; }
                uint32_t r[16];
                tmem_ld16(tmem + TM_O + lane_base + 16 * qt, r);
                tmem_wait_ld();
                float x[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) x[j] = (w0 > 0.f) ? __uint_as_float(r[j]) * w0 : 0.f;
                if (rc.up >= 0) {   // this row lives on in the next stage: leave its fp32 partial there
                    float4 *po = reinterpret_cast<float4 *>(a.part_o + ((size_t)rc.up * H + h) * D + 16 * qt);
#pragma unroll
                    for (int j = 0; j < 4; ++j) po[j] = make_float4(x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]);
                    if (qt == 0) a.part_lse[(size_t)rc.up * H + h] = lse;
                }
                if (qt == 0 && inb) a.lse[(size_t)h * a.T + r0 + rl] = lse;
                uint32_t pk[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) pk[j] = pack_bf16(x[2 * j], x[2 * j + 1]);
                *reinterpret_cast<uint4 *>(sP + rl * 144 + qt * 32) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                *reinterpret_cast<uint4 *>(sP + rl * 144 + qt * 32 + 16) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
            }
            tc_fence_before();
            HDT_STAMP(8);
            __syncthreads();
            HDT_STAMP(10);
            // ---- coalesced stores: thread -> rows tid/8 and tid/8 + 64, 16-byte chunk tid%8 ----
            {
                const int rA = tid >> 3, c = tid & 7;
                __nv_bfloat16 *g = reinterpret_cast<__nv_bfloat16 *>(a.o);
                uint4 v0, v1;
                if (rA < nrows) v0 = *reinterpret_cast<const uint4 *>(sP + rA * 144 + c * 16);
                if (rA + 64 < nrows) v1 = *reinterpret_cast<const uint4 *>(sP + (rA + 64) * 144 + c * 16);
                if (rA < nrows) *reinterpret_cast<uint4 *>(g + ((size_t)(r0 + rA) * H + h) * D + c * 8) = v0;
                if (rA + 64 < nrows) *reinterpret_cast<uint4 *>(g + ((size_t)(r0 + rA + 64) * H + h) * D + c * 8) = v1;
            }
            HDT_STAMP(11);
            dc = dn; dn = dn2; rc = rn;
        }
        if (stamp) {
            for (int i = 0; i < 12; ++i) g_fwd_phase_cycles[i] += ph_acc[i];
            g_fwd_phase_cycles[12] += my_count;
        }
    }
    if (!ok) atomicCAS(a.status, 0, HDT_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TM_COLS);
}
#endif  // HDT_WORKBENCH

// Diagnostics: cycles per phase since the last call; per-CTA timeline of the last instrumented launch.
int read_fwd_timeline(long long *out4096) {
    HDT_CUDA_CHECK(cudaMemcpyFromSymbol(out4096, g_fwd_timeline, sizeof(long long) * 4096));
    return HDT_OK;
}

int read_fwd_phase_cycles(long long *out16) {
    HDT_CUDA_CHECK(cudaMemcpyFromSymbol(out16, g_fwd_phase_cycles, sizeof(long long) * 16));
    long long zero[16] = {0};
    HDT_CUDA_CHECK(cudaMemcpyToSymbol(g_fwd_phase_cycles, zero, sizeof(zero)));
    return HDT_OK;
}

// ---------------------------------------------------------------------------------------------
// Multi-chunk forward at D = 64 for the blocks that are not self-contained (a family longer than
// one block: every block of it walks the whole family's keys in chunks of 128) and for EMPTY
// blocks.  One CTA of 256 threads per (block, head), two CTAs per SM.  Two threads share a query
// row (TMEM lane): thread t and t + 128 take the lower and the upper 64 columns of S, exchange
// their partial row maximum through shared memory and keep partial row sums until the epilogue.
// P goes to TMEM (A operand of the P V MMA); S of chunk i + 1 is issued as soon as every thread
// has S of chunk i in registers (at the barrier of the maximum exchange) and runs beside the
// exponentials, P V of chunk i beside the maximum pass of chunk i + 1; K and V tiles are
// double-buffered; one elected lane of warp 0 requests them, waits for them and issues the MMAs
// inside warp-uniform branches (an MMA issued under a branch on the thread index costs about twice
// the cycles: 100 instead of 40).  The running maximum is only raised when the chunk's maximum
// exceeds it by more than 8 (in the exponent of 2): O and the row sum then need no rescale on
// most chunks, and both use the same reference, so the result is the exact softmax.
// TMEM: S columns [0, 128), O [128, 192), P (bf16 pairs) [192, 256).
// ---------------------------------------------------------------------------------------------
// Cycle counts per phase of k_fwd_tc_mc's chunk loop (STAMP instantiation, option "phase_stamps" =
// 2; read with hdt_debug_fwd_phase_cycles): thread 64 of the eight longest blocks of head 0 adds
// clock64() differences between fixed points of the loop (entries 0 to 6 and 11, chunk count in
// 12), the issuing lane of the same CTAs its waits and issue times (entries 7 to 10).
#define HDT_MSTAMP(i)                                                              \
    do {                                                                           \
        if constexpr (STAMP) {                                                     \
            if (stamper) {                                                         \
                const long long now_ = clock64();                                  \
                atomicAdd((unsigned long long *)&g_fwd_phase_cycles[i], (unsigned long long)(now_ - t_last)); \
                t_last = now_;                                                     \
            }                                                                      \
        }                                                                          \
    } while (0)
template <bool STAMP = false>
__global__ void __launch_bounds__(256, 2) k_fwd_tc_mc(const __grid_constant__ CUtensorMap tm_q,
                                                      const __grid_constant__ CUtensorMap tm_k,
                                                      const __grid_constant__ CUtensorMap tm_v, const FwdStageArgs a) {
    constexpr int D = 64;
    constexpr uint32_t TM_S = 0, TM_O = 128, TM_P = 192, TM_COLS = 256;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = sm;                       // reused to stage O
    uint8_t *sK = sm + SUB;                 // two tiles
    uint8_t *sV = sm + 3 * SUB;             // two tiles
    float *s_x = (float *)(sm + 5 * SUB);   // [2][128]: partial row maxima, at the end partial row sums
    uint64_t *bar_k = (uint64_t *)(s_x + 256);   // [2]; bar_k[0] also carries Q
    uint64_t *bar_v = bar_k + 2;                 // [2]
    uint64_t *bar_s = bar_k + 4, *bar_o = bar_k + 5;   // S of a chunk has arrived; P V of a chunk is done
    uint32_t *slot = (uint32_t *)(bar_k + 6);
    volatile int *abort_flag = (volatile int *)(slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, half = tid >> 7, rl = tid & 127;
    const int blk = a.rest_only ? a.queue_split[a.n_fused + blockIdx.x] : a.queue[blockIdx.x];
    const int h = blockIdx.y, H = a.H;
    const int *rec = a.blocks + 5 * (size_t)blk;
    const int r0 = rec[0], r1 = rec[1], ka = rec[2], kb = rec[3], fl = rec[4];
    const float NEG = -INFINITY, LN2 = 0.6931471805599453f;

    if (tid == 0) {
        for (int i = 0; i < 6; ++i) mbar_init(bar_k + i, 1);
        const int dead0 = (*a.status != 0);
        *abort_flag = dead0;                // an earlier failure: do not wait for anything
        fence_mbar_init();
        // the first tiles are requested before the TMEM allocation and the CTA barrier
        if (!dead0 && !(fl & HDT_BLK_EMPTY) && kb > ka) {
            mbar_expect_tx(bar_k, 2u * SUB);
            tma_load_3d(sQ, &tm_q, 0, h, r0, bar_k);
            tma_load_3d(sK, &tm_k, 0, h, ka, bar_k);
            mbar_expect_tx(bar_v, (uint32_t)SUB);
            tma_load_3d(sV, &tm_v, 0, h, ka, bar_v);
            if (kb - ka > 128) {
                mbar_expect_tx(bar_k + 1, (uint32_t)SUB);
                tma_load_3d(sK + SUB, &tm_k, 0, h, ka + 128, bar_k + 1);
                mbar_expect_tx(bar_v + 1, (uint32_t)SUB);
                tma_load_3d(sV + SUB, &tm_v, 0, h, ka + 128, bar_v + 1);
            }
        }
    }
    if (warp == 0) tmem_alloc(slot, TM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *slot;
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;

    const int row = r0 + rl;
    const bool inb = row < r1;
    int lo = 0, hi = 0;
    if (inb) { lo = a.rng[2 * row]; hi = a.rng[2 * row + 1]; }
    float m = NEG, l = 0.f;
    bool ok = true;
    const bool empty = (fl & HDT_BLK_EMPTY) != 0;
    const bool dead = (*abort_flag != 0);   // same value in every thread: read after the barrier
    const int n_chunks = (empty || dead) ? 0 : (kb - ka + 127) >> 7;
    const float sc = a.scale_log2;

    // S of chunk i: Q K_i^T into TMEM columns [0, 128); thread 0 only
    auto issue_s = [&](int i) {
        const int Nc = (min(128, kb - (ka + 128 * i)) + 15) & ~15;
        const uint32_t idesc = idesc_bf16(Nc, false, false);
        const uint32_t kt = smem_u32(sK + (i & 1) * SUB);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk)
            mma_ss(tmem + TM_S, smem_desc(smem_u32(sQ) + kk * 32, 0, 1024), smem_desc(kt + kk * 32, 0, 1024), idesc, kk > 0);
    };

    if (n_chunks > 0 && warp == 0 && elect_one()) {      // (uniform branch, one lane: the MMA issue is cheaper that way)
        if (!mbar_wait(bar_k, 0, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) a.status[1] = (5 << 8) | 1; }
        if (!*abort_flag) {
            tc_fence_after();
            issue_s(0);
            mma_commit(bar_s);
        }
    }

    long long t_last = 0;
    const bool stamper = STAMP && tid == 64 && blockIdx.y == 0 && blockIdx.x < 8;
    const bool stamp0 = STAMP && blockIdx.y == 0 && blockIdx.x < 8;
    if constexpr (STAMP) { if (stamper) t_last = clock64(); }
    for (int i = 0; i < n_chunks; ++i) {
        const int c0 = ka + 128 * i;
        const int nvalid = min(128, kb - c0);
        const int Nc = (nvalid + 15) & ~15;
        HDT_MSTAMP(11);
        // S of this chunk is there
        if (!mbar_wait(bar_s, i & 1, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) a.status[1] = (5 << 8) | 2; }
        tc_fence_after();
        HDT_MSTAMP(0);
        if (warp == 0 && !*abort_flag && i + 2 < n_chunks && elect_one()) {          // the K tile that S of this chunk has left
            mbar_expect_tx(bar_k + (i & 1), (uint32_t)SUB);
            tma_load_3d(sK + (i & 1) * SUB, &tm_k, 0, h, c0 + 256, bar_k + (i & 1));
        }

        // ---- this thread's 64 columns of S: two slices of 32, all in registers ----
        const int jl = max(lo - c0, 0), jh = min(hi - c0, nvalid);
        const bool has = inb && jh > jl;
        const int cb = 64 * half;
        const bool act0 = cb < Nc, act1 = cb + 32 < Nc;      // uniform in the warp
        uint32_t x0[32], x1[32];
        if (act0) tmem_ld32(tmem + TM_S + lane_base + cb, x0);
        if (act1) tmem_ld32(tmem + TM_S + lane_base + cb + 32, x1);
        if (act0) tmem_wait_ld();
        HDT_MSTAMP(1);
        const uint32_t km0 = (has && act0) ? keep_mask<false>(cb, 32, jl, jh, 0, 0, false, false) : 0u;
        const uint32_t km1 = (has && act1) ? keep_mask<false>(cb + 32, 32, jl, jh, 0, 0, false, false) : 0u;
        const bool full0 = __all_sync(0xffffffffu, km0 == 0xffffffffu);
        const bool full1 = __all_sync(0xffffffffu, km1 == 0xffffffffu);
        float mx = NEG;
        {
            float t0 = NEG, t1 = NEG, t2 = NEG, t3 = NEG;
            if (full0) {
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    t0 = fmaxf(t0, __uint_as_float(x0[j])); t1 = fmaxf(t1, __uint_as_float(x0[j + 1]));
                    t2 = fmaxf(t2, __uint_as_float(x0[j + 2])); t3 = fmaxf(t3, __uint_as_float(x0[j + 3]));
                }
            } else if (km0 != 0u) {
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    t0 = fmaxf(t0, (km0 & (1u << j)) ? __uint_as_float(x0[j]) : NEG);
                    t1 = fmaxf(t1, (km0 & (2u << j)) ? __uint_as_float(x0[j + 1]) : NEG);
                }
            }
            if (full1) {
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    t0 = fmaxf(t0, __uint_as_float(x1[j])); t1 = fmaxf(t1, __uint_as_float(x1[j + 1]));
                    t2 = fmaxf(t2, __uint_as_float(x1[j + 2])); t3 = fmaxf(t3, __uint_as_float(x1[j + 3]));
                }
            } else if (km1 != 0u) {
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    t2 = fmaxf(t2, (km1 & (1u << j)) ? __uint_as_float(x1[j]) : NEG);
                    t3 = fmaxf(t3, (km1 & (2u << j)) ? __uint_as_float(x1[j + 1]) : NEG);
                }
            }
            mx = fmaxf(fmaxf(t0, t1), fmaxf(t2, t3));
        }
        s_x[half * 128 + rl] = mx;
        tc_fence_before();
        __syncthreads();
        HDT_MSTAMP(2);
        // S of the next chunk: every thread holds this chunk's S in registers, so the MMA runs
        // beside the exponentials
        if (warp == 0 && !*abort_flag && i + 1 < n_chunks && elect_one()) {
            tc_fence_after();
            long long t0_ = 0;
            if constexpr (STAMP) t0_ = clock64();
            if (!mbar_wait(bar_k + ((i + 1) & 1), ((i + 1) >> 1) & 1, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) a.status[1] = (5 << 8) | 3; }
            else {
                if constexpr (STAMP) { if (stamp0) { const long long n_ = clock64(); atomicAdd((unsigned long long *)&g_fwd_phase_cycles[7], (unsigned long long)(n_ - t0_)); t0_ = n_; } }
                issue_s(i + 1); mma_commit(bar_s);
                if constexpr (STAMP) { if (stamp0) atomicAdd((unsigned long long *)&g_fwd_phase_cycles[8], (unsigned long long)(clock64() - t0_)); }
            }
        }
        mx = fmaxf(mx, s_x[(half ^ 1) * 128 + rl]);
        // the reference maximum moves only when the chunk's maximum is well above it
        const float mc = mx * sc;
        float alpha = 1.f;
        if (mc > m + 8.f) { alpha = exp2f(m - mc); m = mc; }
        if (i > 0) {          // P V of the previous chunk is done: O may be rescaled, P overwritten, its V tile reused
            if (!mbar_wait(bar_o, (i - 1) & 1, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) a.status[1] = (5 << 8) | 6; }
            tc_fence_after();
            if (warp == 0 && !*abort_flag && i + 1 < n_chunks && elect_one()) {
                mbar_expect_tx(bar_v + ((i + 1) & 1), (uint32_t)SUB);
                tma_load_3d(sV + ((i + 1) & 1) * SUB, &tm_v, 0, h, c0 + 128, bar_v + ((i + 1) & 1));
            }
        }
        HDT_MSTAMP(3);
        if (i > 0 && !__all_sync(0xffffffffu, alpha == 1.f)) {    // rescale this thread's half of the running O
            uint32_t r[32];
            tmem_ld32(tmem + TM_O + lane_base + 32 * half, r);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * alpha);
            tmem_st32(tmem + TM_O + lane_base + 32 * half, r);
        }
        HDT_MSTAMP(4);
        // ---- P = exp2(S scale - m), bf16 pairs into TMEM; partial row sum ----
        float q0 = 0.f, q1 = 0.f, q2 = 0.f, q3 = 0.f;
        if (act0) {
            uint32_t pk[16];
            if (full0) {
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    const float p0 = exp2f(fmaf(__uint_as_float(x0[j]), sc, -m)), p1 = exp2f(fmaf(__uint_as_float(x0[j + 1]), sc, -m));
                    const float p2 = exp2f(fmaf(__uint_as_float(x0[j + 2]), sc, -m)), p3 = exp2f(fmaf(__uint_as_float(x0[j + 3]), sc, -m));
                    q0 += p0; q1 += p1; q2 += p2; q3 += p3;
                    pk[j >> 1] = pack_bf16(p0, p1); pk[(j >> 1) + 1] = pack_bf16(p2, p3);
                }
            } else {
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const float p0 = (km0 & (1u << j)) ? exp2f(fmaf(__uint_as_float(x0[j]), sc, -m)) : 0.f;
                    const float p1 = (km0 & (2u << j)) ? exp2f(fmaf(__uint_as_float(x0[j + 1]), sc, -m)) : 0.f;
                    q0 += p0; q1 += p1;
                    pk[j >> 1] = pack_bf16(p0, p1);
                }
            }
            tmem_st16(tmem + TM_P + lane_base + 32 * half, pk);
        }
        if (act1) {
            uint32_t pk[16];
            if (full1) {
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    const float p0 = exp2f(fmaf(__uint_as_float(x1[j]), sc, -m)), p1 = exp2f(fmaf(__uint_as_float(x1[j + 1]), sc, -m));
                    const float p2 = exp2f(fmaf(__uint_as_float(x1[j + 2]), sc, -m)), p3 = exp2f(fmaf(__uint_as_float(x1[j + 3]), sc, -m));
                    q0 += p0; q1 += p1; q2 += p2; q3 += p3;
                    pk[j >> 1] = pack_bf16(p0, p1); pk[(j >> 1) + 1] = pack_bf16(p2, p3);
                }
            } else {
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const float p0 = (km1 & (1u << j)) ? exp2f(fmaf(__uint_as_float(x1[j]), sc, -m)) : 0.f;
                    const float p1 = (km1 & (2u << j)) ? exp2f(fmaf(__uint_as_float(x1[j + 1]), sc, -m)) : 0.f;
                    q2 += p0; q3 += p1;
                    pk[j >> 1] = pack_bf16(p0, p1);
                }
            }
            tmem_st16(tmem + TM_P + lane_base + 32 * half + 16, pk);
        }
        l = l * alpha + ((q0 + q1) + (q2 + q3));
        tmem_wait_st();
        tc_fence_before();
        HDT_MSTAMP(5);
        __syncthreads();
        HDT_MSTAMP(6);
        if constexpr (STAMP) { if (stamper) atomicAdd((unsigned long long *)&g_fwd_phase_cycles[12], 1ull); }
        if (warp == 0 && !*abort_flag && elect_one()) {
            tc_fence_after();
            long long t0_ = 0;
            if constexpr (STAMP) t0_ = clock64();
            if (!mbar_wait(bar_v + (i & 1), (i >> 1) & 1, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) a.status[1] = (5 << 8) | 4; }
            else {
                if constexpr (STAMP) { if (stamp0) { const long long n_ = clock64(); atomicAdd((unsigned long long *)&g_fwd_phase_cycles[9], (unsigned long long)(n_ - t0_)); t0_ = n_; } }
                const uint32_t idesc = idesc_bf16(D, false, true);
                const uint32_t vt = smem_u32(sV + (i & 1) * SUB);
                const uint64_t dv0 = smem_desc(vt, SUB, 1024);     // the K steps differ in the start address only (16-byte units)
                const int nk16 = Nc / 16;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    if (kk < nk16) mma_ts(tmem + TM_O, tmem + TM_P + 8 * kk, dv0 + (uint64_t)(kk * 128), idesc, (i > 0) || kk > 0);
                mma_commit(bar_o);
                if constexpr (STAMP) { if (stamp0) atomicAdd((unsigned long long *)&g_fwd_phase_cycles[10], (unsigned long long)(clock64() - t0_)); }
            }
        }
    }
    if (n_chunks > 0) {
        if (!mbar_wait(bar_o, (n_chunks - 1) & 1, abort_flag, WAIT_CYCLES)) { ok = false; if (a.status[1] == 0) a.status[1] = (5 << 8) | 5; }
        tc_fence_after();
    }
    if (!ok) atomicCAS(a.status, 0, HDT_ERR_TIMEOUT);

    // ---- epilogue: the row sum is the sum of the two threads' parts; normalise; rows that live on
    // in the next stage also leave their fp32 partial result (O, LSE) there; stage O, store ----
    __syncthreads();                 // the last chunk's maxima have been read
    s_x[half * 128 + rl] = l;
    __syncthreads();
    l = s_x[rl] + s_x[128 + rl];
    float lse = NEG, w0 = 0.f;
    if (l > 0.f) { w0 = 1.f / l; lse = (m + log2f(l)) * LN2; }
    float *po = nullptr;
    if (inb && a.part_o != nullptr) {
        const int u = a.up[row];
        if (u >= 0) {
            po = a.part_o + ((size_t)u * H + h) * D;
            if (half == 0) a.part_lse[(size_t)u * H + h] = lse;
        }
    }
    {
        uint32_t r[32];
        if (n_chunks > 0) {
            tmem_ld32(tmem + TM_O + lane_base + 32 * half, r);
            tmem_wait_ld();
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] = 0u;
        }
        float x[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) x[j] = (w0 > 0.f) ? __uint_as_float(r[j]) * w0 : 0.f;
        if (po != nullptr) {
#pragma unroll
            for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<float4 *>(po + 32 * half + j) = make_float4(x[j], x[j + 1], x[j + 2], x[j + 3]);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c)
            *reinterpret_cast<uint4 *>(sQ + swz(rl, half * 4 + c)) =
                make_uint4(pack_bf16(x[8 * c], x[8 * c + 1]), pack_bf16(x[8 * c + 2], x[8 * c + 3]),
                           pack_bf16(x[8 * c + 4], x[8 * c + 5]), pack_bf16(x[8 * c + 6], x[8 * c + 7]));
    }
    if (inb && half == 0) a.lse[(size_t)h * a.T + row] = lse;
    tc_fence_before();
    __syncthreads();
    {
        __nv_bfloat16 *og = reinterpret_cast<__nv_bfloat16 *>(a.o);
        const int nrows = r1 - r0;
        for (int idx = tid; idx < 128 * 8; idx += 256) {
            const int r = idx >> 3, c = idx & 7;
            if (r < nrows) {
                const uint4 v = *reinterpret_cast<const uint4 *>(sQ + swz(r, c));
                *reinterpret_cast<uint4 *>(og + ((size_t)(r0 + r) * H + h) * D + c * 8) = v;
            }
        }
    }
    if (warp == 0) tmem_dealloc(tmem, TM_COLS);
}

// EMPTY blocks (rows without any key in this stage: PAD, lone roots): zero rows of O, LSE = -inf,
// and the same as partial result of the rows that live on in the next stage.  No shared memory and
// no TMEM, so its CTAs run beside the resident CTAs of the looping kernel (which hold all of an
// SM's TMEM and most of its shared memory).  Blocks of the list that are not EMPTY are skipped.
template <int D>
__global__ void __launch_bounds__(128) k_fwd_empty(const FwdStageArgs a) {
    const int blk = a.rest_only ? a.queue_split[a.n_fused + blockIdx.x] : a.queue[blockIdx.x];
    const int *rec = a.blocks + 5 * (size_t)blk;
    if (!(rec[4] & HDT_BLK_EMPTY)) return;
    const int r0 = rec[0], nrows = rec[1] - r0, h = blockIdx.y, H = a.H;
    __nv_bfloat16 *og = reinterpret_cast<__nv_bfloat16 *>(a.o);
    const uint4 z4 = make_uint4(0u, 0u, 0u, 0u);
    for (int idx = threadIdx.x; idx < nrows * (D / 8); idx += 128) {
        const int r = idx / (D / 8), c = idx % (D / 8);
        *reinterpret_cast<uint4 *>(og + ((size_t)(r0 + r) * H + h) * D + c * 8) = z4;
    }
    for (int r = threadIdx.x; r < nrows; r += 128) {
        const int row = r0 + r;
        a.lse[(size_t)h * a.T + row] = -INFINITY;
        if (a.part_o != nullptr) {
            const int u = a.up[row];
            if (u >= 0) {
                float4 *po = reinterpret_cast<float4 *>(a.part_o + ((size_t)u * H + h) * D);
                for (int j = 0; j < D / 4; ++j) po[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                a.part_lse[(size_t)u * H + h] = -INFINITY;
            }
        }
    }
}

template <int D>
static int launch_fwd_tc_t(const FwdStageArgs &a, cudaStream_t st) {
    CUtensorMap tq, tk, tv;
    int rc = make_tmap_bf16(&tq, a.q, D, a.H, a.T, 128);
    if (rc) return rc;
    rc = make_tmap_bf16(&tk, a.k, D, a.H, a.T, 128);
    if (rc) return rc;
    rc = make_tmap_bf16(&tv, a.v, D, a.H, a.T, 128);
    if (rc) return rc;
    OutMaps om;      // the looping kernel's output tiles leave through TMA stores (boxes of 64 .. 1 rows)
    for (int bx = 0; bx < 7; ++bx) {
        rc = make_tmap_bf16(&om.m[bx], a.o, D, a.H, a.T, 64 >> bx);
        if (rc) return rc;
    }
    constexpr int smem = (4 * (D / 64) + 2) * SUB + 1024 + 64;     // general kernel: Q, two K tiles, V, P
    constexpr int smem_1 = 3 * (D / 64) * SUB + 1024 + 64;
    constexpr int smem_mc = 5 * SUB + 2 * 128 * 4 + 1024 + 64;     // multi-chunk kernel: Q, two K, two V tiles
    static DevOnce attr;
    if (!attr.done()) {
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_fwd_tc<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_fwd_tc<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_1));
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_fwd_tc_loop<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_1));
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_fwd_tc_loop<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_1));
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_fwd_tc<D, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_fwd_tc_mc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_mc));
#ifdef HDT_WORKBENCH
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_fwd_tc_p, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            8 * SUB + 4 * 128 * 4 + 1024 + 64));
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_fwd_tc_mc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_mc));
#endif
        attr.set();
    }
    const bool dirs = a.dirs != 7;   // direction bits: the instantiations that apply them
    if (a.hdr != nullptr) {          // counts on the device only: the looping kernel with all its CTAs
        int n_sm_e = 0;
        if (const int rc_ = sm_count(&n_sm_e)) return rc_;
        const int grid = n_sm_e * (D == 64 ? 4 : 2);
        if (dirs) k_fwd_tc_loop<D, true><<<grid, 128, smem_1, st>>>(tq, tk, tv, om, a);
        else k_fwd_tc_loop<D><<<grid, 128, smem_1, st>>>(tq, tk, tv, om, a);
        count_launch();
        HDT_CUDA_CHECK(cudaGetLastError());
        return HDT_OK;
    }
    FwdStageArgs b = a;
    b.rest_only = 0;
    int n_general = a.nb;
    const bool split_launch = a.no_persistent != 1;     // two kernels: self-contained blocks, the others
    if (a.n_fused > 0 && split_launch && a.part == 2) {  // the caller launches the looping kernel separately
        b.rest_only = 1;
        n_general = a.nb - a.n_fused;
    } else if (a.n_fused > 0 && split_launch) {
#ifdef HDT_WORKBENCH
        if (D == 64 && a.no_persistent == 2 && !dirs) {   // option: the persistent single-CTA-per-SM kernel
            constexpr int smem_p = 8 * SUB + 4 * 128 * 4 + 1024 + 64;
            int n_sm = 0;
            if (const int rc_ = sm_count(&n_sm)) return rc_;
            const long long items = (long long)a.n_fused * a.H;
            k_fwd_tc_p<<<(int)(items < n_sm ? items : n_sm), 512, smem_p, st>>>(tq, tk, tv, a);
        } else
#endif
        if (a.no_persistent == 3 && !dirs) {       // option: one CTA per (block, head), no loop
            k_fwd_tc<D, true><<<dim3(a.n_fused, a.H), 128, smem_1, st>>>(tq, tk, tv, a);
        } else {
            int n_sm = 0;
            if (const int rc_ = sm_count(&n_sm)) return rc_;
            const long long items = (long long)a.n_fused * a.H;
            const long long slots = (long long)n_sm * (D == 64 ? 4 : 2);
            if (dirs) k_fwd_tc_loop<D, true><<<(int)(items < slots ? items : slots), 128, smem_1, st>>>(tq, tk, tv, om, a);
#ifdef HDT_WORKBENCH
            else if (g_phase_stamps == 1 && D == 64) {
                static DevOnce attr_s;
                if (!attr_s.done()) {
                    HDT_CUDA_CHECK(cudaFuncSetAttribute(k_fwd_tc_loop<64, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_1));
                    attr_s.set();
                }
                k_fwd_tc_loop<64, false, true><<<(int)(items < slots ? items : slots), 128, 3 * SUB + 1024 + 64, st>>>(tq, tk, tv, om, a);
            }
#endif
            else k_fwd_tc_loop<D><<<(int)(items < slots ? items : slots), 128, smem_1, st>>>(tq, tk, tv, om, a);
        }
        count_launch();
        HDT_CUDA_CHECK(cudaGetLastError());
        b.rest_only = 1;
        n_general = a.nb - a.n_fused;
    }
    if (a.part == 1 && split_launch) n_general = 0;     // the caller launches the other blocks separately
    if (n_general > 0) {
        dim3 grid(n_general, a.H);
        if (a.n_empty == n_general && !g_no_fwd_mc) k_fwd_empty<D><<<grid, 128, 0, st>>>(b);   // nothing but EMPTY blocks left
        else if (dirs) k_fwd_tc<D, false, false, true><<<grid, 128, smem, st>>>(tq, tk, tv, b);
#ifdef HDT_WORKBENCH
        else if (D == 64 && !g_no_fwd_mc && g_phase_stamps == 2) k_fwd_tc_mc<true><<<grid, 256, smem_mc, st>>>(tq, tk, tv, b);
#endif
        else if (D == 64 && !g_no_fwd_mc) k_fwd_tc_mc<false><<<grid, 256, smem_mc, st>>>(tq, tk, tv, b);
        else k_fwd_tc<D, false><<<grid, 128, smem, st>>>(tq, tk, tv, b);
        count_launch();
        HDT_CUDA_CHECK(cudaGetLastError());
    }
    return HDT_OK;
}

// A stage above 0 in own-partial mode (a.tok and a.own_* set): one CTA per (block, head).
template <int D>
static int launch_fwd_tc_upper_t(const FwdStageArgs &a, cudaStream_t st) {
    CUtensorMap tq;     // the gathering kernel takes no tensor map; the parameter slots get a valid one
    int rc = make_tmap_bf16(&tq, a.q, D, a.H, a.T, 128);
    if (rc) return rc;
    constexpr int smem = (3 * (D / 64) + 2) * SUB + 1024 + 64;
    static DevOnce attr;
    if (!attr.done()) {
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_fwd_tc<D, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_fwd_tc<D, false, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attr.set();
    }
    FwdStageArgs b = a;
    b.rest_only = 0;
    if (a.dirs != 7) {      // direction bits: the general layout's instantiation that applies them
        k_fwd_tc<D, false, true, true><<<dim3(a.nb, a.H), 128, smem, st>>>(tq, tq, tq, b);
        count_launch();
        HDT_CUDA_CHECK(cudaGetLastError());
        return HDT_OK;
    }
    // every block self-contained (keys = its own rows, one chunk): the single-chunk layout (P over the
    // Q / K tiles, O over S) needs 48 KB and 128 TMEM columns at D = 64, so four CTAs share an SM
    // instead of two and the stage runs in one wave
    if (a.n_fused == a.nb && a.queue_split != nullptr && !g_no_fwd_mc) {
        constexpr int smem_1 = 3 * (D / 64) * SUB + 1024 + 64;
        static DevOnce attr_1;
        if (!attr_1.done()) {
            HDT_CUDA_CHECK(cudaFuncSetAttribute(k_fwd_tc<D, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_1));
            attr_1.set();
        }
        k_fwd_tc<D, true, true><<<dim3(a.nb, a.H), 128, smem_1, st>>>(tq, tq, tq, b);
    } else
        k_fwd_tc<D, false, true><<<dim3(a.nb, a.H), 128, smem, st>>>(tq, tq, tq, b);
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;
}

int launch_fwd_tc_upper(const FwdStageArgs &a, int D, cudaStream_t st) {
    if (a.nb == 0) return HDT_OK;
    if (a.tok == nullptr || (!a.final_merge && (a.own_o == nullptr || a.own_lse == nullptr)) ||
        (a.final_merge == 1 && (a.carry_o == nullptr || a.carry_lse == nullptr)) ||
        (a.final_merge == 2 && (a.carry_o != nullptr || a.next_own_o != nullptr || a.o == nullptr || a.lse == nullptr)))
        return set_error(HDT_ERR_INVALID_ARG, "launch_fwd_tc_upper: needs a tok map and own-partial (or carry) buffers");
    if (D == 64) return launch_fwd_tc_upper_t<64>(a, st);
    if (D == 128) return launch_fwd_tc_upper_t<128>(a, st);
    return set_error(HDT_ERR_UNSUPPORTED, "head_dim %d not supported (64 or 128)", D);
}

int launch_fwd_tc(const FwdStageArgs &a, int D, cudaStream_t st) {
    if (a.nb == 0 && a.hdr == nullptr) return HDT_OK;
    if (D == 64) return launch_fwd_tc_t<64>(a, st);
    if (D == 128) return launch_fwd_tc_t<128>(a, st);
    return set_error(HDT_ERR_UNSUPPORTED, "head_dim %d not supported (64 or 128)", D);
}

}  // namespace hdt
