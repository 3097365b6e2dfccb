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

template <int D>
__global__ void __launch_bounds__(128) k_fwd_tc(const __grid_constant__ CUtensorMap tm_q,
                                                const __grid_constant__ CUtensorMap tm_k,
                                                const __grid_constant__ CUtensorMap tm_v, const FwdStageArgs a) {
    constexpr int NSUB = D / 64;
    constexpr uint32_t TM_S = 0, TM_O = 128, TM_COLS = 256;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sQ = sm;                       // NSUB sub-tiles; reused to stage O
    uint8_t *sK = sQ + NSUB * SUB;
    uint8_t *sV = sK + NSUB * SUB;
    uint8_t *sP = sV + NSUB * SUB;          // 2 sub-tiles (128 keys)
    uint64_t *bar_tma = (uint64_t *)(sP + 2 * SUB);
    uint64_t *bar_mma = bar_tma + 1;
    uint32_t *slot = (uint32_t *)(bar_mma + 1);
    volatile int *abort_flag = (volatile int *)(slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5;
    const int blk = a.queue[blockIdx.x], h = blockIdx.y, H = a.H;
    const int *rec = a.blocks + 5 * (size_t)blk;
    const int r0 = rec[0], r1 = rec[1], ka = rec[2], kb = rec[3], fl = rec[4];
    const float NEG = -INFINITY, LN2 = 0.6931471805599453f;

    if (tid == 0) {
        mbar_init(bar_tma, 1);
        mbar_init(bar_mma, 1);
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
    const bool empty = (fl & HDT_BLK_EMPTY) != 0;
    const bool dead = (*abort_flag != 0);   // same value in every thread: read after the barrier

    if (!empty && !dead) {
        for (int c0 = ka; c0 < kb; c0 += 128) {
            const int nvalid = min(128, kb - c0);
            const int Nc = (nvalid + 15) & ~15;
            const bool first = (c0 == ka);
            if (tid == 0 && !*abort_flag) {   // after a failed wait nothing new is issued
                mbar_expect_tx(bar_tma, (uint32_t)((first ? NSUB : 0) + 2 * NSUB) * SUB);
                for (int s = 0; s < NSUB; ++s) {
                    if (first) tma_load_3d(sQ + s * SUB, &tm_q, 64 * s, h, r0, bar_tma);
                    tma_load_3d(sK + s * SUB, &tm_k, 64 * s, h, c0, bar_tma);
                    tma_load_3d(sV + s * SUB, &tm_v, 64 * s, h, c0, bar_tma);
                }
            }
            ok = mbar_wait(bar_tma, ph_tma, abort_flag, WAIT_CYCLES) && ok;
            ph_tma ^= 1;
            if (tid == 0 && !*abort_flag) {
                tc_fence_after();
                const uint32_t idesc = idesc_bf16(Nc, false, false);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk / 4) * SUB + (kk % 4) * 32;
                    mma_ss(tmem + TM_S, smem_desc(smem_u32(sQ) + off, 0, 1024), smem_desc(smem_u32(sK) + off, 0, 1024),
                           idesc, kk > 0);
                }
                mma_commit(bar_mma);
            }
            ok = mbar_wait(bar_mma, ph_mma, abort_flag, WAIT_CYCLES) && ok;
            ph_mma ^= 1;
            tc_fence_after();

            // ---- masked online softmax of this row over the chunk's columns ----
            const int jl = max(lo - c0, 0), jh = min(hi - c0, nvalid);
            const bool has = inb && jh > jl;
            const int nsl = (Nc + 31) >> 5;
            float mx = NEG;
            for (int k = 0; k < nsl; ++k) {
                const int s0 = 32 * k;
                const bool mine = has && jl < s0 + 32 && jh > s0;
                if (__any_sync(0xffffffffu, mine)) {
                    uint32_t r[32];
                    tmem_ld32(tmem + TM_S + lane_base + s0, r);
                    tmem_wait_ld();
                    if (mine) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (s0 + j >= jl && s0 + j < jh) mx = fmaxf(mx, __uint_as_float(r[j]));
                    }
                }
            }
            const float m_new = fmaxf(m, mx * a.scale_log2);
            const float alpha = (m_new == NEG) ? 1.f : exp2f(m - m_new);
            float lsum = 0.f;
            for (int k = 0; k < nsl; ++k) {
                const int s0 = 32 * k;
                const bool mine = has && jl < s0 + 32 && jh > s0;
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
                            if (s0 + j >= jl && s0 + j < jh) p0 = exp2f(fmaf(__uint_as_float(r[j]), a.scale_log2, -m_new));
                            if (s0 + j + 1 >= jl && s0 + j + 1 < jh)
                                p1 = exp2f(fmaf(__uint_as_float(r[j + 1]), a.scale_log2, -m_new));
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
            ok = mbar_wait(bar_mma, ph_mma, abort_flag, WAIT_CYCLES) && ok;
            ph_mma ^= 1;
            tc_fence_after();
        }
    }
    if (!ok && tid == 0) atomicCAS(a.status, 0, HDT_ERR_TIMEOUT);

    // ---- epilogue: normalise; rows that live on in the next stage also leave their fp32 partial
    // result (O, LSE) there, the next stage completes and overwrites them; stage O, store ----
    float lse = NEG, w0 = 0.f;
    if (l > 0.f) { w0 = 1.f / l; lse = (m + log2f(l)) * LN2; }
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

template <int D>
static int launch_fwd_tc_t(const FwdStageArgs &a, cudaStream_t st) {
    CUtensorMap tq, tk, tv;
    int rc = make_tmap_bf16(&tq, a.q, D, a.H, a.T, 128);
    if (rc) return rc;
    rc = make_tmap_bf16(&tk, a.k, D, a.H, a.T, 128);
    if (rc) return rc;
    rc = make_tmap_bf16(&tv, a.v, D, a.H, a.T, 128);
    if (rc) return rc;
    constexpr int smem = (3 * (D / 64) + 2) * SUB + 1024 + 64;
    static bool attr = false;
    if (!attr) {
        HDT_CUDA_CHECK(cudaFuncSetAttribute(k_fwd_tc<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attr = true;
    }
    dim3 grid(a.nb, a.H);
    k_fwd_tc<D><<<grid, 128, smem, st>>>(tq, tk, tv, a);
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;
}

int launch_fwd_tc(const FwdStageArgs &a, int D, cudaStream_t st) {
    if (a.nb == 0) return HDT_OK;
    if (D == 64) return launch_fwd_tc_t<64>(a, st);
    if (D == 128) return launch_fwd_tc_t<128>(a, st);
    return set_error(HDT_ERR_UNSUPPORTED, "head_dim %d not supported (64 or 128)", D);
}

}  // namespace hdt
