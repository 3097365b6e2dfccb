// FP32 SIMT attention kernels over the staged family index.
//
// These are the exact-arithmetic path: fp32 inputs (where tensor cores have no fp32-input
// mode accurate to 1e-4) and the small compacted stages above stage 0 (a few percent of the
// tokens).  One CTA handles one (row block, head); a row is owned by G = D/16 adjacent lanes,
// each holding 16 of the D dimensions; keys/values of the block's span are staged through
// shared memory in chunks and every row walks only its own key range [lo, hi).
#include <cuda_bf16.h>

#include "hdt_internal.cuh"

namespace hdt {

static constexpr int KC = 32;        // keys per shared-memory chunk

template <bool BF16>
__device__ __forceinline__ float4 load4(const void *base, size_t elem) {
    if constexpr (BF16) {
        const uint2 u = *reinterpret_cast<const uint2 *>(reinterpret_cast<const __nv_bfloat16 *>(base) + elem);
        float4 r;
        r.x = __uint_as_float(u.x << 16);
        r.y = __uint_as_float(u.x & 0xffff0000u);
        r.z = __uint_as_float(u.y << 16);
        r.w = __uint_as_float(u.y & 0xffff0000u);
        return r;
    } else {
        return *reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(base) + elem);
    }
}

template <bool BF16>
__device__ __forceinline__ void store4(void *base, size_t elem, float4 v) {
    if constexpr (BF16) {
        __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
        uint2 u;
        u.x = *reinterpret_cast<uint32_t *>(&a);
        u.y = *reinterpret_cast<uint32_t *>(&b);
        *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(base) + elem) = u;
    } else {
        *reinterpret_cast<float4 *>(reinterpret_cast<float *>(base) + elem) = v;
    }
}

__device__ __forceinline__ float dot4(float4 a, float4 b, float acc) {
    acc = fmaf(a.x, b.x, acc);
    acc = fmaf(a.y, b.y, acc);
    acc = fmaf(a.z, b.z, acc);
    acc = fmaf(a.w, b.w, acc);
    return acc;
}
__device__ __forceinline__ void axpy4(float4 &y, float a, float4 x) {
    y.x = fmaf(a, x.x, y.x);
    y.y = fmaf(a, x.y, y.y);
    y.z = fmaf(a, x.z, y.z);
    y.w = fmaf(a, x.w, y.w);
}
__device__ __forceinline__ void scale4(float4 &y, float a) { y.x *= a; y.y *= a; y.z *= a; y.w *= a; }

template <int G>
__device__ __forceinline__ float group_sum(float x) {
    x += __shfl_xor_sync(0xffffffffu, x, 1);
    x += __shfl_xor_sync(0xffffffffu, x, 2);
    if constexpr (G == 8) x += __shfl_xor_sync(0xffffffffu, x, 4);
    return x;
}

// Stage `rows` [c0, c0+KC) of a [*, H, D] tensor (through tok) into smem as fp32, zero past `end`.
template <int D, bool BF16, int NTHREADS>
__device__ __forceinline__ void stage_rows(float4 *dst, const void *src, const int *tok, int c0, int end,
                                           int H, int h) {
    constexpr int U = D / 4;
    for (int idx = threadIdx.x; idx < KC * U; idx += NTHREADS) {
        const int r = idx / U, u = idx % U;
        const int e = c0 + r;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (e < end) {
            const int t = tok ? tok[e] : e;
            v = load4<BF16>(src, ((size_t)t * H + h) * D + 4 * u);
        }
        dst[idx] = v;
    }
}

// ---------------------------------------------------------------------------------------------
// forward
// ---------------------------------------------------------------------------------------------
// (the body for entry bx of a stage's queue: the one-stage kernel and the kernel over several stages call it)
template <int D, bool BF16, int NTHREADS>
__device__ __forceinline__ void fwd_simt_block(const FwdStageArgs &a, int bx) {
    constexpr int G = D / 16, U = D / 4, RP = NTHREADS / G;
    __shared__ float4 sK[KC * U];
    __shared__ float4 sV[KC * U];
    const int blk = a.queue[bx], h = blockIdx.y, H = a.H;
    const int *rec = a.blocks + 5 * (size_t)blk;
    const int r0 = rec[0], r1 = rec[1], ka = rec[2], kb = rec[3];
    const int g = threadIdx.x % G, rl = threadIdx.x / G;
    const float NEG = -INFINITY;

    for (int p0 = r0; p0 < r1; p0 += RP) {
        const int row = p0 + rl;
        const bool inb = row < r1;
        int lo = 0, hi = 0, trow = 0;
        float4 q[4], o[4];
#pragma unroll
        for (int t = 0; t < 4; ++t) { q[t] = make_float4(0, 0, 0, 0); o[t] = make_float4(0, 0, 0, 0); }
        if (inb) {
            lo = a.rng[2 * row];
            hi = a.rng[2 * row + 1];
            trow = a.tok_rows ? a.tok_rows[row] : row;
#pragma unroll
            for (int t = 0; t < 4; ++t) q[t] = load4<BF16>(a.q, ((size_t)trow * H + h) * D + 4 * (g + G * t));
        }
        float m = NEG, l = 0.f;
        for (int c0 = ka; c0 < kb; c0 += KC) {
            __syncthreads();
            stage_rows<D, BF16, NTHREADS>(sK, a.k, a.tok, c0, kb, H, h);
            stage_rows<D, BF16, NTHREADS>(sV, a.v, a.tok, c0, kb, H, h);
            __syncthreads();
            const int jlo = max(lo, c0), jhi = min(hi, c0 + KC);
            const bool has = jhi > jlo;
            const int wlo = __reduce_min_sync(0xffffffffu, has ? jlo : 0x7fffffff);
            const int whi = __reduce_max_sync(0xffffffffu, has ? jhi : (int)0x80000000);
            for (int j0 = wlo; j0 < whi; j0 += 8) {
                float s[8];
#pragma unroll
                for (int jj = 0; jj < 8; ++jj) {
                    const int j = j0 + jj;
                    s[jj] = NEG;
                    if (j < whi) {
                        const float4 *kr = sK + (j - c0) * U;
                        float acc = 0.f;
#pragma unroll
                        for (int t = 0; t < 4; ++t) acc = dot4(q[t], kr[g + G * t], acc);
                        acc = group_sum<G>(acc);
                        if (j >= jlo && j < jhi && (a.dirs == 7 || dir_ok(row, j, lo, a.dirs))) s[jj] = acc * a.scale_log2;
                    }
                }
                float mx = s[0];
#pragma unroll
                for (int jj = 1; jj < 8; ++jj) mx = fmaxf(mx, s[jj]);
                const float mn = fmaxf(m, mx);
                if (mn > NEG) {
                    const float alpha = exp2f(m - mn);
                    l *= alpha;
#pragma unroll
                    for (int t = 0; t < 4; ++t) scale4(o[t], alpha);
#pragma unroll
                    for (int jj = 0; jj < 8; ++jj) {
                        const int j = j0 + jj;
                        if (j < whi) {
                            const float p = exp2f(s[jj] - mn);
                            l += p;
                            const float4 *vr = sV + (j - c0) * U;
#pragma unroll
                            for (int t = 0; t < 4; ++t) axpy4(o[t], p, vr[g + G * t]);
                        }
                    }
                    m = mn;
                }
            }
        }
        if (!inb) continue;
        // own partial result, natural-log LSE
        float lse = NEG;
        if (l > 0.f) {
            const float inv = 1.f / l;
#pragma unroll
            for (int t = 0; t < 4; ++t) scale4(o[t], inv);
            lse = (m + log2f(l)) * 0.6931471805599453f;
        }
        if (a.own_o != nullptr) {   // computed beside stage 0: leave the own partial, merge later
            float4 *po = reinterpret_cast<float4 *>(a.own_o + ((size_t)row * H + h) * D);
#pragma unroll
            for (int t = 0; t < 4; ++t) po[g + G * t] = o[t];
            if (g == 0) a.own_lse[(size_t)row * H + h] = lse;
            continue;
        }
        // merge the partial result the stages below left for this element (same index)
        if (a.carry_o != nullptr) {
            const float lc = a.carry_lse[(size_t)row * H + h];
            if (lc > NEG) {
                const float mx = fmaxf(lse, lc);
                const float e0 = (lse > NEG) ? __expf(lse - mx) : 0.f, e1 = __expf(lc - mx);
                const float tot = e0 + e1;
                const float w0 = e0 / tot, w1 = e1 / tot;
                const float4 *oc = reinterpret_cast<const float4 *>(a.carry_o + ((size_t)row * H + h) * D);
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    scale4(o[t], w0);
                    axpy4(o[t], w1, oc[g + G * t]);
                }
                lse = mx + __logf(tot);
            }
        }
        // hand the merged partial to the next stage if the element lives on there ...
        const int u = (a.part_o != nullptr) ? a.up[row] : -1;
        if (u >= 0) {
            float4 *po = reinterpret_cast<float4 *>(a.part_o + ((size_t)u * H + h) * D);
#pragma unroll
            for (int t = 0; t < 4; ++t) po[g + G * t] = o[t];
            if (g == 0) a.part_lse[(size_t)u * H + h] = lse;
        }
        // ... and write the result so far; a later stage overwrites it with the complete one
#pragma unroll
        for (int t = 0; t < 4; ++t) store4<BF16>(a.o, ((size_t)trow * H + h) * D + 4 * (g + G * t), o[t]);
        if (g == 0) a.lse[(size_t)h * a.T + trow] = lse;
    }
}

template <int D, bool BF16, int NTHREADS>
__global__ void __launch_bounds__(NTHREADS) k_fwd_simt(const FwdStageArgs a) {
    fwd_simt_block<D, BF16, NTHREADS>(a, (int)blockIdx.x);
}
// Several stages in own-partial mode (deep trees: a launch per stage is mostly launch latency) in one
// launch: CTA x belongs to the stage s with cum[s] <= x < cum[s + 1] and is entry x - cum[s] of its queue.
template <int D, bool BF16, int NTHREADS>
__global__ void __launch_bounds__(NTHREADS) k_fwd_simt_multi(const MultiFwdArgs m) {
    int s = 0;
    while (s + 1 < m.n && (int)blockIdx.x >= m.st[s + 1].cum) ++s;
    FwdStageArgs a = m.base;
    const MultiStage &t = m.st[s];
    a.n = t.n; a.nb = t.nb; a.tok = t.tok; a.tok_rows = t.tok; a.rng = t.rng; a.up = t.up; a.blocks = t.blocks; a.queue = t.queue;
    a.own_o = t.own[0]; a.own_lse = t.own_lse;
    fwd_simt_block<D, BF16, NTHREADS>(a, (int)blockIdx.x - t.cum);
}

// ---------------------------------------------------------------------------------------------
// backward: phase A rows -> dQ, phase B keys -> dK, dV (the family ranges are symmetric, so the
// same blocks serve as key blocks)
// ---------------------------------------------------------------------------------------------
template <int D, bool BF16, int NTHREADS>
__device__ __forceinline__ void bwd_simt_block(const BwdStageArgs &a, int bx) {
    constexpr int G = D / 16, U = D / 4, RP = NTHREADS / G;
    __shared__ float4 sA[KC * U];  // K (phase A) / Q (phase B)
    __shared__ float4 sB[KC * U];  // V (phase A) / dO (phase B)
    __shared__ float sL[KC], sDl[KC];
    const int blk = a.queue[bx], h = blockIdx.y, H = a.H;
    const int *rec = a.blocks + 5 * (size_t)blk;
    const int r0 = rec[0], r1 = rec[1], ka = rec[2], kb = rec[3];
    const int g = threadIdx.x % G, rl = threadIdx.x / G;
    const float LOG2E = 1.4426950408889634f;

    for (int p0 = r0; p0 < r1; p0 += RP) {
        const int row = p0 + rl;
        const bool inb = row < r1;
        int lo = 0, hi = 0, trow = 0;
        if (inb) {
            lo = a.rng[2 * row];
            hi = a.rng[2 * row + 1];
            trow = a.tok_rows ? a.tok_rows[row] : row;
        }
        const bool live = hi > lo;
        // ---------------- phase A: this element as a query row ----------------
        float4 x[4], y[4], acc[4];  // q, dO, dq
        if (a.phases != 2) {   // same decision in the whole grid
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            x[t] = y[t] = acc[t] = make_float4(0, 0, 0, 0);
            if (live) {
                x[t] = load4<BF16>(a.q, ((size_t)trow * H + h) * D + 4 * (g + G * t));
                y[t] = load4<BF16>(a.d_o, ((size_t)trow * H + h) * D + 4 * (g + G * t));
            }
        }
        float lse2 = 0.f, dl = 0.f;
        if (live) {
            lse2 = a.lse[(size_t)h * a.T + trow] * LOG2E;
            dl = a.delta[(size_t)h * a.T + trow];
        }
        for (int c0 = ka; c0 < kb; c0 += KC) {
            __syncthreads();
            stage_rows<D, BF16, NTHREADS>(sA, a.k, a.tok, c0, kb, H, h);
            stage_rows<D, BF16, NTHREADS>(sB, a.v, a.tok, c0, kb, H, h);
            __syncthreads();
            const int jlo = max(lo, c0), jhi = min(hi, c0 + KC);
            const bool has = jhi > jlo;
            const int wlo = __reduce_min_sync(0xffffffffu, has ? jlo : 0x7fffffff);
            const int whi = __reduce_max_sync(0xffffffffu, has ? jhi : (int)0x80000000);
            for (int j = wlo; j < whi; ++j) {
                const float4 *kr = sA + (j - c0) * U, *vr = sB + (j - c0) * U;
                float s = 0.f, dp = 0.f;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    s = dot4(x[t], kr[g + G * t], s);
                    dp = dot4(y[t], vr[g + G * t], dp);
                }
                s = group_sum<G>(s);
                dp = group_sum<G>(dp);
                if (j >= jlo && j < jhi && (a.dirs == 7 || dir_ok(row, j, lo, a.dirs))) {
                    const float p = exp2f(s * a.scale_log2 - lse2);
                    const float ds = p * (dp - dl);
#pragma unroll
                    for (int t = 0; t < 4; ++t) axpy4(acc[t], ds, kr[g + G * t]);
                }
            }
        }
        if (inb && a.own_dq != nullptr) {
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                scale4(acc[t], a.scale);
                reinterpret_cast<float4 *>(a.own_dq + ((size_t)row * H + h) * D)[g + G * t] = acc[t];
            }
        } else if (inb) {
            const int u = (a.part_dq != nullptr) ? a.up[row] : -1;
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                scale4(acc[t], a.scale);
                if (a.carry_dq != nullptr) {   // partial gradient from the stages below (same index)
                    const float4 c = reinterpret_cast<const float4 *>(a.carry_dq + ((size_t)row * H + h) * D)[g + G * t];
                    acc[t].x += c.x; acc[t].y += c.y; acc[t].z += c.z; acc[t].w += c.w;
                }
                if (u >= 0) reinterpret_cast<float4 *>(a.part_dq + ((size_t)u * H + h) * D)[g + G * t] = acc[t];
                store4<BF16>(a.dq, ((size_t)trow * H + h) * D + 4 * (g + G * t), acc[t]);
            }
        }
        }
        if (a.phases == 1) continue;
        // ---------------- phase B: this element as a key ----------------
        float4 acc2[4];  // x = k, y = v, acc = dk, acc2 = dv
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            x[t] = y[t] = acc[t] = acc2[t] = make_float4(0, 0, 0, 0);
            if (live) {
                x[t] = load4<BF16>(a.k, ((size_t)trow * H + h) * D + 4 * (g + G * t));
                y[t] = load4<BF16>(a.v, ((size_t)trow * H + h) * D + 4 * (g + G * t));
            }
        }
        for (int c0 = ka; c0 < kb; c0 += KC) {
            __syncthreads();
            stage_rows<D, BF16, NTHREADS>(sA, a.q, a.tok, c0, kb, H, h);
            stage_rows<D, BF16, NTHREADS>(sB, a.d_o, a.tok, c0, kb, H, h);
            if (threadIdx.x < KC) {   // KC <= NTHREADS
                const int e = c0 + threadIdx.x;
                float L = 0.f, dlt = 0.f;
                if (e < kb) {
                    const int t = a.tok ? a.tok[e] : e;
                    L = a.lse[(size_t)h * a.T + t] * LOG2E;
                    dlt = a.delta[(size_t)h * a.T + t];
                }
                sL[threadIdx.x] = L;
                sDl[threadIdx.x] = dlt;
            }
            __syncthreads();
            const int jlo = max(lo, c0), jhi = min(hi, c0 + KC);
            const bool has = jhi > jlo;
            const int wlo = __reduce_min_sync(0xffffffffu, has ? jlo : 0x7fffffff);
            const int whi = __reduce_max_sync(0xffffffffu, has ? jhi : (int)0x80000000);
            for (int i = wlo; i < whi; ++i) {
                const float4 *qr = sA + (i - c0) * U, *dor = sB + (i - c0) * U;
                float s = 0.f, dp = 0.f;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    s = dot4(x[t], qr[g + G * t], s);
                    dp = dot4(y[t], dor[g + G * t], dp);
                }
                s = group_sum<G>(s);
                dp = group_sum<G>(dp);
                if (i >= jlo && i < jhi && (a.dirs == 7 || dir_ok_key(row, i, lo, a.dirs))) {
                    const float p = exp2f(s * a.scale_log2 - sL[i - c0]);
                    const float ds = p * (dp - sDl[i - c0]);
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        axpy4(acc[t], ds, qr[g + G * t]);
                        axpy4(acc2[t], p, dor[g + G * t]);
                    }
                }
            }
        }
        if (inb && a.own_dq != nullptr) {
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                scale4(acc[t], a.scale);
                reinterpret_cast<float4 *>(a.own_dk + ((size_t)row * H + h) * D)[g + G * t] = acc[t];
                reinterpret_cast<float4 *>(a.own_dv + ((size_t)row * H + h) * D)[g + G * t] = acc2[t];
            }
        } else if (inb) {
            const int u = (a.part_dk != nullptr) ? a.up[row] : -1;
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                scale4(acc[t], a.scale);
                if (a.carry_dk != nullptr) {
                    const float4 c = reinterpret_cast<const float4 *>(a.carry_dk + ((size_t)row * H + h) * D)[g + G * t];
                    const float4 c2 = reinterpret_cast<const float4 *>(a.carry_dv + ((size_t)row * H + h) * D)[g + G * t];
                    acc[t].x += c.x; acc[t].y += c.y; acc[t].z += c.z; acc[t].w += c.w;
                    acc2[t].x += c2.x; acc2[t].y += c2.y; acc2[t].z += c2.z; acc2[t].w += c2.w;
                }
                if (u >= 0) {
                    reinterpret_cast<float4 *>(a.part_dk + ((size_t)u * H + h) * D)[g + G * t] = acc[t];
                    reinterpret_cast<float4 *>(a.part_dv + ((size_t)u * H + h) * D)[g + G * t] = acc2[t];
                }
                store4<BF16>(a.dk, ((size_t)trow * H + h) * D + 4 * (g + G * t), acc[t]);
                store4<BF16>(a.dv, ((size_t)trow * H + h) * D + 4 * (g + G * t), acc2[t]);
            }
        }
    }
}

template <int D, bool BF16, int NTHREADS>
__global__ void __launch_bounds__(NTHREADS) k_bwd_simt(const BwdStageArgs a) {
    bwd_simt_block<D, BF16, NTHREADS>(a, (int)blockIdx.x);
}
template <int D, bool BF16, int NTHREADS>
__global__ void __launch_bounds__(NTHREADS) k_bwd_simt_multi(const MultiBwdArgs m) {
    int s = 0;
    while (s + 1 < m.n && (int)blockIdx.x >= m.st[s + 1].cum) ++s;
    BwdStageArgs a = m.base;
    const MultiStage &t = m.st[s];
    a.n = t.n; a.nb = t.nb; a.tok = t.tok; a.tok_rows = t.tok; a.rng = t.rng; a.up = t.up; a.blocks = t.blocks; a.queue = t.queue;
    a.own_dq = t.own[0]; a.own_dk = t.own[1]; a.own_dv = t.own[2];
    bwd_simt_block<D, BF16, NTHREADS>(a, (int)blockIdx.x - t.cum);
}

// delta[h, t] = sum_c dO[t,h,c] * O[t,h,c].  A (token, head) row is read by LPR adjacent lanes with
// one 16-byte load each per tensor (8 bf16 or 4 fp32 values), so a warp covers 32 / LPR rows.
template <int D, bool BF16>
__global__ void __launch_bounds__(256) k_delta(const void *o, const void *d_o, float *delta, int T, int H) {
    constexpr int VPL = BF16 ? 8 : 4;          // values per lane
    constexpr int LPR = D / VPL;               // lanes per row: 8 (bf16, D=64) ... 32 (fp32, D=128)
    const long long gtid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long row = gtid / LPR;
    const int sub = (int)(gtid % LPR);
    float acc = 0.f;
    if (row < (long long)T * H) {
        if constexpr (BF16) {
            const uint4 x = *reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(o) + row * D + sub * 8);
            const uint4 y = *reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(d_o) + row * D + sub * 8);
            const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                acc = fmaf(__uint_as_float(xs[i] << 16), __uint_as_float(ys[i] << 16), acc);
                acc = fmaf(__uint_as_float(xs[i] & 0xffff0000u), __uint_as_float(ys[i] & 0xffff0000u), acc);
            }
        } else {
            const float4 x = *reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(o) + row * D + sub * 4);
            const float4 y = *reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(d_o) + row * D + sub * 4);
            acc = dot4(x, y, 0.f);
        }
    }
#pragma unroll
    for (int s = LPR / 2; s; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
    if (sub == 0 && row < (long long)T * H) {
        const int t = (int)(row / H), h = (int)(row % H);
        delta[(size_t)h * T + t] = acc;
    }
}

// ---------------------------------------------------------------------------------------------
// Completion of the tokens that live in stages above 0, after those stages were computed beside
// stage 0 (one thread per 4 values of a (stage-1 element, head)).
// ---------------------------------------------------------------------------------------------
template <int D, bool BF16>
__global__ void __launch_bounds__(256) k_chain_merge(const ChainArgs c) {
    constexpr int U = D / 4;
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long rowh = gid / U;           // stage-1 element * H + head
    const int u4 = (int)(gid % U);
    if (rowh >= (long long)c.n1 * c.H) return;
    const int e1 = (int)(rowh / c.H), h = (int)(rowh % c.H);
    const int t = c.tok1[e1];
    const float NEG = -INFINITY;
    if (c.nt == 1) {   // forward: log-sum-exp merge
        float lse = c.base_lse[rowh];
        float4 o = reinterpret_cast<const float4 *>(c.base[0] + rowh * D)[u4];
        int e = e1;
        for (int s = 1; s < c.n_stages; ++s) {
            const size_t r = (size_t)e * c.H + h;
            const float lc = c.own_lse[s][r];
            if (lc > NEG) {
                const float mx = fmaxf(lse, lc);
                const float w0 = (lse > NEG) ? __expf(lse - mx) : 0.f, w1 = __expf(lc - mx);
                const float tot = w0 + w1;
                const float4 oc = reinterpret_cast<const float4 *>(c.own[s][0] + r * D)[u4];
                scale4(o, w0 / tot);
                axpy4(o, w1 / tot, oc);
                lse = mx + __logf(tot);
            }
            e = c.up[s][e];
            if (e < 0) break;
        }
        store4<BF16>(c.out[0], ((size_t)t * c.H + h) * D + 4 * u4, o);
        if (u4 == 0) c.lse[(size_t)h * c.T + t] = lse;
    } else {           // backward: sums
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            float4 x = reinterpret_cast<const float4 *>(c.base[k] + rowh * D)[u4];
            int e = e1;
            for (int s = 1; s < c.n_stages; ++s) {
                const float4 y = reinterpret_cast<const float4 *>(c.own[s][k] + ((size_t)e * c.H + h) * D)[u4];
                x.x += y.x; x.y += y.y; x.z += y.z; x.w += y.w;
                e = c.up[s][e];
                if (e < 0) break;
            }
            store4<BF16>(c.out[k], ((size_t)t * c.H + h) * D + 4 * u4, x);
        }
    }
}

template <int D, bool BF16>
static int launch_chain_t(const ChainArgs &c, cudaStream_t st) {
    const long long threads = (long long)c.n1 * c.H * (D / 4);
    if (threads == 0) return HDT_OK;
    k_chain_merge<D, BF16><<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(c);
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;
}
int launch_chain_merge(const ChainArgs &c, int D, int dtype, cudaStream_t st) {
    if (D == 64) return dtype == HDT_BF16 ? launch_chain_t<64, true>(c, st) : launch_chain_t<64, false>(c, st);
    if (D == 128) return dtype == HDT_BF16 ? launch_chain_t<128, true>(c, st) : launch_chain_t<128, false>(c, st);
    return set_error(HDT_ERR_UNSUPPORTED, "head_dim %d not supported (64 or 128)", D);
}

// Small row blocks (the stages above 0) run with 128-thread CTAs so that several fit on an SM.
template <int D, bool BF16>
static int launch_fwd_t(const FwdStageArgs &a, cudaStream_t st) {
    if (a.nb == 0) return HDT_OK;
    dim3 grid(a.nb, a.H);
    if (a.block_rows <= 32) k_fwd_simt<D, BF16, 128><<<grid, 128, 0, st>>>(a);
    else k_fwd_simt<D, BF16, 512><<<grid, 512, 0, st>>>(a);
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;
}
template <int D, bool BF16>
static int launch_bwd_t(const BwdStageArgs &a, cudaStream_t st) {
    if (a.nb == 0) return HDT_OK;
    dim3 grid(a.nb, a.H);
    if (a.block_rows <= 32) k_bwd_simt<D, BF16, 128><<<grid, 128, 0, st>>>(a);
    else k_bwd_simt<D, BF16, 512><<<grid, 512, 0, st>>>(a);
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;
}

template <int D, bool BF16>
static int launch_fwd_multi_t(const MultiFwdArgs &m, cudaStream_t st) {
    const int total = m.st[m.n - 1].cum + m.st[m.n - 1].nb;
    if (total == 0) return HDT_OK;
    dim3 grid(total, m.base.H);
    if (m.base.block_rows <= 32) k_fwd_simt_multi<D, BF16, 128><<<grid, 128, 0, st>>>(m);
    else k_fwd_simt_multi<D, BF16, 512><<<grid, 512, 0, st>>>(m);
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;
}
template <int D, bool BF16>
static int launch_bwd_multi_t(const MultiBwdArgs &m, cudaStream_t st) {
    const int total = m.st[m.n - 1].cum + m.st[m.n - 1].nb;
    if (total == 0) return HDT_OK;
    dim3 grid(total, m.base.H);
    if (m.base.block_rows <= 32) k_bwd_simt_multi<D, BF16, 128><<<grid, 128, 0, st>>>(m);
    else k_bwd_simt_multi<D, BF16, 512><<<grid, 512, 0, st>>>(m);
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;
}
int launch_fwd_simt_multi(const MultiFwdArgs &m, int D, int dtype, cudaStream_t st) {
    if (m.n <= 0) return HDT_OK;
    if (D == 64) return dtype == HDT_BF16 ? launch_fwd_multi_t<64, true>(m, st) : launch_fwd_multi_t<64, false>(m, st);
    if (D == 128) return dtype == HDT_BF16 ? launch_fwd_multi_t<128, true>(m, st) : launch_fwd_multi_t<128, false>(m, st);
    return set_error(HDT_ERR_UNSUPPORTED, "head_dim %d not supported (64 or 128)", D);
}
int launch_bwd_simt_multi(const MultiBwdArgs &m, int D, int dtype, cudaStream_t st) {
    if (m.n <= 0) return HDT_OK;
    if (D == 64) return dtype == HDT_BF16 ? launch_bwd_multi_t<64, true>(m, st) : launch_bwd_multi_t<64, false>(m, st);
    if (D == 128) return dtype == HDT_BF16 ? launch_bwd_multi_t<128, true>(m, st) : launch_bwd_multi_t<128, false>(m, st);
    return set_error(HDT_ERR_UNSUPPORTED, "head_dim %d not supported (64 or 128)", D);
}

int launch_fwd_simt(const FwdStageArgs &a, int D, int dtype, cudaStream_t st) {
    if (D == 64) return dtype == HDT_BF16 ? launch_fwd_t<64, true>(a, st) : launch_fwd_t<64, false>(a, st);
    if (D == 128) return dtype == HDT_BF16 ? launch_fwd_t<128, true>(a, st) : launch_fwd_t<128, false>(a, st);
    return set_error(HDT_ERR_UNSUPPORTED, "head_dim %d not supported (64 or 128)", D);
}
int launch_bwd_simt(const BwdStageArgs &a, int D, int dtype, cudaStream_t st) {
    if (D == 64) return dtype == HDT_BF16 ? launch_bwd_t<64, true>(a, st) : launch_bwd_t<64, false>(a, st);
    if (D == 128) return dtype == HDT_BF16 ? launch_bwd_t<128, true>(a, st) : launch_bwd_t<128, false>(a, st);
    return set_error(HDT_ERR_UNSUPPORTED, "head_dim %d not supported (64 or 128)", D);
}

template <int D, bool BF16>
static void launch_delta_t(const void *o, const void *d_o, float *delta, int T, int H, cudaStream_t st) {
    constexpr int LPR = D / (BF16 ? 8 : 4);
    const long long threads = (long long)T * H * LPR;
    k_delta<D, BF16><<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(o, d_o, delta, T, H);
}

int launch_delta(const void *o, const void *d_o, float *delta, int T, int H, int D, int dtype, cudaStream_t st) {
    if ((long long)T * H == 0) return HDT_OK;
    if (D == 64) {
        if (dtype == HDT_BF16) launch_delta_t<64, true>(o, d_o, delta, T, H, st);
        else launch_delta_t<64, false>(o, d_o, delta, T, H, st);
    } else if (D == 128) {
        if (dtype == HDT_BF16) launch_delta_t<128, true>(o, d_o, delta, T, H, st);
        else launch_delta_t<128, false>(o, d_o, delta, T, H, st);
    } else {
        return set_error(HDT_ERR_UNSUPPORTED, "head_dim %d not supported (64 or 128)", D);
    }
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;
}

}  // namespace hdt
