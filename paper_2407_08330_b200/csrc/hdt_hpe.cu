// Hierarchical positional encoding (paper, paragraph "Hierarchical Positional Encoding", the
// positional-encoding equation): every token has one index p^l per hierarchy level l = 1..L (the
// number of its level-l ancestor among that ancestor's siblings, counted from 1; 0 on the levels
// below an anchor's own level and for the root), and
//     HPE(p, 2k) = sum_l sin(w_k p^l),  HPE(p, 2k+1) = sum_l cos(w_k p^l),  w_k = 10000^(-2k/d_model).
// The sibling numbers come for free from the staged index: in the stage where a node is handled as
// a child of its family, its number is its distance from the family head; the index build writes it
// (hdt_index::rank) where it finds the family.
#include <cuda_bf16.h>

#include "hdt_internal.cuh"
#include "hdt_sm100.cuh"

namespace hdt {

// pvec[token, l-1] = p^l: walk up from the token, one ancestor per level
__global__ void k_hpe_pvec(const int8_t *__restrict__ level, const int32_t *__restrict__ parent,
                           const int32_t *__restrict__ cu, int B, int T, int L, const int *__restrict__ rank,
                           int *pvec) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= T) return;
    int lo = 0, hi = B;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (cu[mid] <= i) lo = mid; else hi = mid;
    }
    const int s0 = cu[lo];
    for (int l = 0; l < L; ++l) pvec[(size_t)i * L + l] = 0;
    int node = i, lv = level[i];
    while (lv >= 1) {          // PAD (-1) and the root (0) keep all zeros
        if (lv <= L) pvec[(size_t)i * L + (lv - 1)] = rank[node];
        node = s0 + parent[node];
        --lv;
    }
}

// One thread per (frequency k, token chunk).  The angle w_k p is formed and reduced to [-pi, pi] in
// double (p reaches thousands, w_0 = 1), the sine and cosine of the reduced angle in float.
template <bool BF16>
__global__ void __launch_bounds__(128) k_hpe_eval(const int8_t *__restrict__ level, const int *__restrict__ pvec, int T,
                                                  int L, int d_model, int accumulate, int tokens_per_cta, void *x) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    const int half = d_model >> 1;
    if (k >= half) return;
    const double w = exp2(-2.0 * (double)k / (double)d_model * 13.287712379549449 /* log2(10000) */);
    const double inv2pi = 0.15915494309189535, twopi = 6.283185307179586;
    const int t0 = blockIdx.y * tokens_per_cta, t1 = min(T, t0 + tokens_per_cta);
    for (int t = t0; t < t1; ++t) {
        float s = 0.f, c = 0.f;
        if (level[t] >= 0) {
            for (int l = 0; l < L; ++l) {
                const double th = w * (double)pvec[(size_t)t * L + l];
                const float r = (float)(th - twopi * rint(th * inv2pi));
                float sn, cs;
                __sincosf(r, &sn, &cs);
                s += sn;
                c += cs;
            }
        }
        const size_t off = (size_t)t * d_model + 2 * k;
        if constexpr (BF16) {
            __nv_bfloat162 *p = reinterpret_cast<__nv_bfloat162 *>(reinterpret_cast<__nv_bfloat16 *>(x) + off);
            if (accumulate) {
                const float2 o = __bfloat1622float2(*p);
                s += o.x;
                c += o.y;
            }
            *p = __floats2bfloat162_rn(s, c);
        } else {
            float2 *p = reinterpret_cast<float2 *>(reinterpret_cast<float *>(x) + off);
            if (accumulate) {
                const float2 o = *p;
                s += o.x;
                c += o.y;
            }
            *p = make_float2(s, c);
        }
    }
}

// Vector form for d_model % 8 == 0: a thread owns 4 consecutive frequencies (8 outputs, 16 bytes of
// bf16 or 32 bytes of fp32) and a run of consecutive tokens.  The angle w_k p is carried as an
// unevaluated float pair (w_k = wh + wl, product error recovered with fma) and reduced by 2 pi in
// two steps, which keeps it within a few 1e-7 for p < 2^20.  Tokens of one sentence share the
// section and sentence numbers, so a level's sine and cosine are recomputed only when its p changes.
constexpr int HPE_TOK = 4;   // tokens loaded together (independent 16/32-byte loads in flight)

template <bool BF16, int L>
__global__ void __launch_bounds__(384, 2) k_hpe_eval_vec(const int8_t *__restrict__ level, const int *__restrict__ pvec,
                                                      int t_begin, int T, int Lrt, int d_model, int accumulate,
                                                      int run, void *x) {
    const int G = d_model >> 3;
    const int nl = L ? L : Lrt;
    const int chunk0 = t_begin + (blockIdx.x * blockDim.y + threadIdx.y) * run;
    const int t_end = min(T, chunk0 + run);
    if (chunk0 >= T) return;
    for (int g = threadIdx.x; g < G; g += blockDim.x) {
        float wh[4], wl[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const double w = exp2(-2.0 * (double)(4 * g + j) / (double)d_model * 13.287712379549449 /* log2(10000) */);
            wh[j] = (float)w;
            wl[j] = (float)(w - (double)wh[j]);
        }
        constexpr int LC = L ? L : 1;
        int pc[LC];                 // cached p per level (compile-time L only)
        float sc[LC][4], cc[LC][4];
#pragma unroll
        for (int l = 0; l < LC; ++l) {
            pc[l] = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) { sc[l][j] = 0.f; cc[l][j] = 1.f; }
        }
        for (int t0 = chunk0; t0 < t_end; t0 += HPE_TOK) {
            constexpr int NV = BF16 ? 1 : 2;          // 16-byte vectors per thread and token
            uint4 raw[HPE_TOK][NV];
            int lv[HPE_TOK], pv[HPE_TOK][LC];
#pragma unroll
            for (int u = 0; u < HPE_TOK; ++u) {
                const int t = t0 + u;
                lv[u] = t < t_end ? (int)level[t] : -1;
                if constexpr (L > 0) {      // all loads of the group are issued before any arithmetic
#pragma unroll
                    for (int l = 0; l < L; ++l) pv[u][l] = t < t_end ? pvec[(size_t)t * L + l] : 0;
                }
#pragma unroll
                for (int i = 0; i < NV; ++i) raw[u][i] = make_uint4(0u, 0u, 0u, 0u);   // +0.0 in either type
                if (accumulate && t < t_end) {
                    const uint4 *src = reinterpret_cast<const uint4 *>(
                        reinterpret_cast<const char *>(x) + ((size_t)t * d_model + 8 * g) * (BF16 ? 2 : 4));
#pragma unroll
                    for (int i = 0; i < NV; ++i) raw[u][i] = src[i];
                }
            }
#pragma unroll
            for (int u = 0; u < HPE_TOK; ++u) {
                const int t = t0 + u;
                if (t >= t_end) break;
                float s[4] = {0.f, 0.f, 0.f, 0.f}, c[4] = {0.f, 0.f, 0.f, 0.f};
                if (lv[u] >= 0) {
#pragma unroll
                    for (int l = 0; l < nl; ++l) {
                        const int lc = L ? l : 0;
                        const int p = L ? pv[u][lc] : pvec[(size_t)t * nl + l];
                        if (!L || p != pc[lc]) {
                            const float pf = (float)p;
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const float th = pf * wh[j];
                                const float tl = fmaf(pf, wl[j], fmaf(pf, wh[j], -th));
                                const float n = rintf(th * 0.15915494309189535f);
                                float r = fmaf(-n, 6.2831854820251465f, th);       // 2 pi rounded to float
                                r = fmaf(n, 1.7484555e-7f, r) + tl;                // ... minus what that rounding added
                                __sincosf(r, &sc[lc][j], &cc[lc][j]);
                            }
                            pc[lc] = p;
                        }
#pragma unroll
                        for (int j = 0; j < 4; ++j) { s[j] += sc[lc][j]; c[j] += cc[lc][j]; }
                    }
                }
                uint4 *dst = reinterpret_cast<uint4 *>(
                    reinterpret_cast<char *>(x) + ((size_t)t * d_model + 8 * g) * (BF16 ? 2 : 4));
                if constexpr (BF16) {
                    uint4 r = raw[u][0];
                    __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&r);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float2 f = __bfloat1622float2(h[j]);
                        h[j] = __floats2bfloat162_rn(f.x + s[j], f.y + c[j]);
                    }
                    dst[0] = r;
                } else {
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        float4 f = *reinterpret_cast<float4 *>(&raw[u][i]);
                        f.x += s[2 * i]; f.y += c[2 * i]; f.z += s[2 * i + 1]; f.w += c[2 * i + 1];
                        dst[i] = *reinterpret_cast<uint4 *>(&f);
                    }
                }
            }
        }
    }
}

// x += HPE(p) as a bulk-copy pipeline (d_model % 8 == 0, three levels): a resident CTA walks tiles
// of HPE_R tokens; one thread keeps up to HPE_NS - 1 tiles of x rows, p-vectors and levels in
// flight as bulk copies into shared memory, the CTA adds the encoding in place there and the same
// thread sends the tile back with a bulk store.  Thread (g, y) owns frequencies 4g..4g+3 of the
// HPE_R / 4 consecutive tokens y * HPE_R / 4 ... of each tile.  Along such a run the section and
// sentence numbers rarely change and the token number mostly grows by one, so the thread keeps
// the sum of the first two levels, re-evaluates a sine/cosine only for a level whose p changed,
// and advances the third level by the rotation (sin, cos)(a + w) from (sin, cos)(a) and
// (sin, cos)(w) when p grew by exactly one.  A run is at most HPE_R / 4 tokens long and restarts
// from a full evaluation, so the rotations add at most a few 1e-7 of error.
constexpr int HPE_R = 32, HPE_NS = 4;     // tokens per tile; most stages a CTA keeps

// (sin, cos)(p w) with p w carried as a float pair and reduced by 2 pi in two steps
__device__ __forceinline__ void hpe_sincos(float pf, float wh, float wl, float &sn, float &cs) {
    const float th = pf * wh;
    const float tl = fmaf(pf, wl, fmaf(pf, wh, -th));
    const float n = __fadd_rn(__fadd_rn(th * 0.15915494309189535f, 12582912.f), -12582912.f);   // nearest integer
    float a = fmaf(-n, 6.2831854820251465f, th);          // 2 pi rounded to float ...
    a = fmaf(n, 1.7484555e-7f, a) + tl;                   // ... minus what that rounding added
    __sincosf(a, &sn, &cs);
}

template <bool BF16>
__global__ void __launch_bounds__(512, 1) k_hpe_acc_bulk(const int8_t *__restrict__ level, const int *__restrict__ pvec,
                                                         int n_tiles, int d_model, int ns, void *x, int *status) {
    using namespace sm100;
    constexpr int L = 3, ESZ = BF16 ? 2 : 4, NV = BF16 ? 1 : 2, TPT = HPE_R / 4;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ uint64_t full[HPE_NS];
    __shared__ int abort_flag;
    const uint32_t row_bytes = (uint32_t)d_model * ESZ;
    const uint32_t x_bytes = HPE_R * row_bytes, p_bytes = HPE_R * L * 4, l_bytes = HPE_R;
    const uint32_t stage_bytes = x_bytes + p_bytes + l_bytes;        // multiple of 16
    const int tid = threadIdx.y * blockDim.x + threadIdx.x;
    if (tid == 0) {
        for (int i = 0; i < HPE_NS; ++i) mbar_init(&full[i], 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    const int n_mine = blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    auto issue = [&](int i) {       // thread 0: fetch my i-th tile into stage i % ns
        const int tile = blockIdx.x + i * gridDim.x;
        unsigned char *st = smem + (size_t)(i % ns) * stage_bytes;
        uint64_t *bar = &full[i % ns];
        mbar_expect_tx(bar, stage_bytes);
        bulk_load(st, reinterpret_cast<const char *>(x) + (size_t)tile * x_bytes, x_bytes, bar);
        bulk_load(st + x_bytes, pvec + (size_t)tile * HPE_R * L, p_bytes, bar);
        bulk_load(st + x_bytes + p_bytes, level + (size_t)tile * HPE_R, l_bytes, bar);
    };
    if (tid == 0)
        for (int i = 0; i < ns - 1 && i < n_mine; ++i) issue(i);

    const int G = d_model >> 3, g = threadIdx.x;      // blockDim.x >= G: one frequency group per thread
    float wh[4], wl[4], sw[4], cw[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const double w = exp2(-2.0 * (double)(4 * g + j) / (double)d_model * 13.287712379549449 /* log2(10000) */);
        wh[j] = (float)w;
        wl[j] = (float)(w - (double)wh[j]);
        __sincosf(wh[j], &sw[j], &cw[j]);             // w <= 1: no reduction needed
    }
    for (int i = 0; i < n_mine; ++i) {
        unsigned char *st = smem + (size_t)(i % ns) * stage_bytes;
        if (!mbar_wait(&full[i % ns], (i / ns) & 1, &abort_flag, 2000000000LL)) break;
        const int *sp = reinterpret_cast<const int *>(st + x_bytes);
        const int8_t *sl = reinterpret_cast<const int8_t *>(st + x_bytes + p_bytes);
        if (g < G) {
            // p = 0 on every level: sin 0 = 0, cos 0 = 1
            int pc0 = 0, pc1 = 0, pc2 = 0;
            float s0[4], c0[4], s1[4], c1[4], s2[4], c2[4], bs[4], bc[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                s0[j] = s1[j] = s2[j] = 0.f;
                c0[j] = c1[j] = c2[j] = 1.f;
                bs[j] = 0.f;
                bc[j] = 2.f;
            }
#pragma unroll 2
            for (int u = 0; u < TPT; ++u) {
                const int r = threadIdx.y * TPT + u;
                if (sl[r] < 0) continue;                    // PAD rows pass through unchanged
                const int p0 = sp[r * L], p1 = sp[r * L + 1], p2 = sp[r * L + 2];
                if (p0 != pc0 || p1 != pc1) {
                    if (p0 != pc0) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) hpe_sincos((float)p0, wh[j], wl[j], s0[j], c0[j]);
                        pc0 = p0;
                    }
                    if (p1 != pc1) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) hpe_sincos((float)p1, wh[j], wl[j], s1[j], c1[j]);
                        pc1 = p1;
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) { bs[j] = s0[j] + s1[j]; bc[j] = c0[j] + c1[j]; }
                }
                if (p2 == pc2 + 1) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float sn = fmaf(s2[j], cw[j], c2[j] * sw[j]);
                        c2[j] = fmaf(c2[j], cw[j], -s2[j] * sw[j]);
                        s2[j] = sn;
                    }
                } else if (p2 != pc2) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) hpe_sincos((float)p2, wh[j], wl[j], s2[j], c2[j]);
                }
                pc2 = p2;
                uint4 *cell = reinterpret_cast<uint4 *>(st + (size_t)r * row_bytes + (size_t)g * 8 * ESZ);
                if constexpr (BF16) {
                    uint4 v = cell[0];
                    __nv_bfloat162 *h = reinterpret_cast<__nv_bfloat162 *>(&v);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float2 f = __bfloat1622float2(h[j]);
                        h[j] = __floats2bfloat162_rn(f.x + (bs[j] + s2[j]), f.y + (bc[j] + c2[j]));
                    }
                    cell[0] = v;
                } else {
#pragma unroll
                    for (int q = 0; q < NV; ++q) {
                        float4 f = *reinterpret_cast<float4 *>(&cell[q]);
                        f.x += bs[2 * q] + s2[2 * q];
                        f.y += bc[2 * q] + c2[2 * q];
                        f.z += bs[2 * q + 1] + s2[2 * q + 1];
                        f.w += bc[2 * q + 1] + c2[2 * q + 1];
                        cell[q] = *reinterpret_cast<uint4 *>(&f);
                    }
                }
            }
        }
        fence_proxy_async_smem();       // the tile was written through the generic proxy
        __syncthreads();
        if (tid == 0) {
            const int tile = blockIdx.x + i * gridDim.x;
            bulk_store(reinterpret_cast<char *>(x) + (size_t)tile * x_bytes, st, x_bytes);
            bulk_commit();
            if (i + ns - 1 < n_mine) {
                bulk_wait_read_1();     // the stage refilled next was stored one tile ago
                issue(i + ns - 1);
            }
        }
    }
    if (tid == 0) {
        bulk_wait_all();
        if (abort_flag) atomicCAS(status, 0, (int)HDT_ERR_TIMEOUT);
    }
}

}  // namespace hdt

using namespace hdt;

static size_t al256h(size_t v) { return (v + 255) & ~size_t(255); }

extern "C" size_t hdt_hpe_workspace_bytes(const hdt_index_t *ix, int32_t n_levels) {
    if (!ix || n_levels < 1 || n_levels > 32) return 0;
    const size_t T = (size_t)ix->total_tokens;
    return al256h(sizeof(int) * T * n_levels) + 256;
}

extern "C" int hdt_hpe(const hdt_index_t *ix, const int8_t *level, const int32_t *parent, const int32_t *cu_seqlens,
                       int32_t n_levels, int32_t d_model, int32_t dtype, int32_t accumulate, void *x,
                       void *workspace, size_t workspace_bytes, void *stream) {
    if (!ix) return set_error(HDT_ERR_INVALID_ARG, "hdt_hpe: null index");
    if (const int rc0 = index_ready(ix)) return rc0;
    if (n_levels < 1 || n_levels > 32 || d_model < 2 || (d_model & 1))
        return set_error(HDT_ERR_INVALID_ARG, "hdt_hpe: n_levels must be 1..32, d_model even and positive");
    if (dtype != HDT_F32 && dtype != HDT_BF16) return set_error(HDT_ERR_UNSUPPORTED, "hdt_hpe: unknown dtype %d", dtype);
    const int T = ix->total_tokens, B = ix->batch;
    if (T == 0) return HDT_OK;
    if (!level || !parent || !cu_seqlens || !x) return set_error(HDT_ERR_INVALID_ARG, "hdt_hpe: null pointer");
    const size_t need = hdt_hpe_workspace_bytes(ix, n_levels);
    if (!workspace || workspace_bytes < need)
        return set_error(HDT_ERR_WORKSPACE, "hdt_hpe: workspace %zu < required %zu", workspace_bytes, need);
    if (((uintptr_t)workspace & 255) || ((uintptr_t)x & 7))
        return set_error(HDT_ERR_INVALID_ARG, "hdt_hpe: workspace must be 256-byte, x 8-byte aligned");
    cudaStream_t st = (cudaStream_t)stream;
    const int *rank = ix->rank;
    int *pvec = (int *)workspace;
    k_hpe_pvec<<<(T + 255) / 256, 256, 0, st>>>(level, parent, cu_seqlens, B, T, n_levels, rank, pvec);
    count_launch();
    const bool x16 = ((uintptr_t)x & 15) == 0;
    if (d_model % 8 == 0 && x16) {
        // threads.x covers the 8-element groups of a row (whole warps), threads.y token runs
        const int G = d_model / 8;
        int t_begin = 0;
        const size_t esz = dtype == HDT_BF16 ? 2 : 4;
        const size_t stage = (size_t)HPE_R * d_model * esz + HPE_R * 3 * 4 + HPE_R;
        const int ns = (int)min((size_t)HPE_NS, (size_t)(220 * 1024) / stage);
        if (accumulate && n_levels == 3 && G <= 128 && ns >= 2 && T >= HPE_R && ((uintptr_t)level & 15) == 0) {
            // whole tiles through the bulk-copy pipeline, the ragged tail through the register kernel
            const int n_tiles = T / HPE_R;
            const int tx = ((G + 31) / 32) * 32;
            const size_t smem = stage * ns;
            const int per_sm = (int)max((size_t)1, min((size_t)2, (size_t)(220 * 1024) / (smem + 1024)));
            const int nb = min(n_tiles, 148 * per_sm);
            int *status = device_status_ptr();
            static DevOnce attr_done;
            if (!attr_done.done()) {
                HDT_CUDA_CHECK(cudaFuncSetAttribute(k_hpe_acc_bulk<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
                HDT_CUDA_CHECK(cudaFuncSetAttribute(k_hpe_acc_bulk<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024));
                attr_done.set();
            }
            if (dtype == HDT_BF16) k_hpe_acc_bulk<true><<<nb, dim3(tx, 4), smem, st>>>(level, pvec, n_tiles, d_model, ns, x, status);
            else k_hpe_acc_bulk<false><<<nb, dim3(tx, 4), smem, st>>>(level, pvec, n_tiles, d_model, ns, x, status);
            count_launch();
            t_begin = n_tiles * HPE_R;
        }
        if (t_begin < T) {
        const int tx = min(384, ((G + 31) / 32) * 32), ty = max(1, 384 / tx);
        int run = 16;
        const int Tr = T - t_begin;
        while ((long long)((Tr + run - 1) / run + ty - 1) / ty > 148LL * 64) run *= 2;
        const int nb = ((Tr + run - 1) / run + ty - 1) / ty;
        const dim3 blk(tx, ty);
#define HPE_LAUNCH(BF, LL) k_hpe_eval_vec<BF, LL><<<nb, blk, 0, st>>>(level, pvec, t_begin, T, n_levels, d_model, accumulate, run, x)
        if (dtype == HDT_BF16) {
            if (n_levels == 3) HPE_LAUNCH(true, 3); else if (n_levels == 2) HPE_LAUNCH(true, 2); else HPE_LAUNCH(true, 0);
        } else {
            if (n_levels == 3) HPE_LAUNCH(false, 3); else if (n_levels == 2) HPE_LAUNCH(false, 2); else HPE_LAUNCH(false, 0);
        }
        count_launch();
        }
#undef HPE_LAUNCH
    } else {
        const int half = d_model / 2;
        const int gx = (half + 127) / 128;
        int tokens_per_cta = 32;
        while ((long long)gx * ((T + tokens_per_cta - 1) / tokens_per_cta) > 65535LL * 4 && tokens_per_cta < (1 << 20)) tokens_per_cta *= 2;
        const dim3 grid(gx, (T + tokens_per_cta - 1) / tokens_per_cta);
        if (grid.y > 65535) return set_error(HDT_ERR_UNSUPPORTED, "hdt_hpe: too many tokens");
        if (dtype == HDT_BF16) k_hpe_eval<true><<<grid, 128, 0, st>>>(level, pvec, T, n_levels, d_model, accumulate, tokens_per_cta, x);
        else k_hpe_eval<false><<<grid, 128, 0, st>>>(level, pvec, T, n_levels, d_model, accumulate, tokens_per_cta, x);
        count_launch();
    }
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;
}
