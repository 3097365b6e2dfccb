// Hierarchical positional encoding (paper, paragraph "Hierarchical Positional Encoding", the
// positional-encoding equation): every token has one index p^l per hierarchy level l = 1..L (the
// number of its level-l ancestor among that ancestor's siblings, counted from 1; 0 on the levels
// below an anchor's own level and for the root), and
//     HPE(p, 2k) = sum_l sin(w_k p^l),  HPE(p, 2k+1) = sum_l cos(w_k p^l),  w_k = 10000^(-2k/d_model).
// The sibling numbers come for free from the staged index: in the stage where a node is handled as
// a child of its family, its number is its distance from the family head.
#include <cuda_bf16.h>

#include "hdt_internal.cuh"

namespace hdt {

// rank[token] = sibling number (1-based) of every element that is a family child in this stage
__global__ void k_hpe_rank(int n, const int *__restrict__ tok, const int *__restrict__ par,
                           const int *__restrict__ rng, int *rank) {
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const int lo = rng[2 * e], hi = rng[2 * e + 1], p = par[e];
        if (hi > lo && p >= 0 && lo == p) rank[tok[e]] = e - lo;
    }
}

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

}  // namespace hdt

using namespace hdt;

static size_t al256h(size_t v) { return (v + 255) & ~size_t(255); }

extern "C" size_t hdt_hpe_workspace_bytes(const hdt_index_t *ix, int32_t n_levels) {
    if (!ix || n_levels < 1 || n_levels > 32) return 0;
    const size_t T = (size_t)ix->total_tokens;
    return al256h(sizeof(int) * T) + al256h(sizeof(int) * T * n_levels) + 256;
}

extern "C" int hdt_hpe(const hdt_index_t *ix, const int8_t *level, const int32_t *parent, const int32_t *cu_seqlens,
                       int32_t n_levels, int32_t d_model, int32_t dtype, int32_t accumulate, void *x,
                       void *workspace, size_t workspace_bytes, void *stream) {
    if (!ix) return set_error(HDT_ERR_INVALID_ARG, "hdt_hpe: null index");
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
    int *rank = (int *)workspace;
    int *pvec = (int *)((char *)workspace + al256h(sizeof(int) * (size_t)T));
    HDT_CUDA_CHECK(cudaMemsetAsync(rank, 0, sizeof(int) * (size_t)T, st));
    for (int s = 0; s < ix->n_stages; ++s) {
        const int n = ix->desc[s].n;
        if (n == 0) continue;
        const StagePtrs &P = ix->st[s];
        k_hpe_rank<<<min((n + 255) / 256, 148 * 8), 256, 0, st>>>(n, P.tok, P.par, P.rng, rank);
        count_launch();
    }
    k_hpe_pvec<<<(T + 255) / 256, 256, 0, st>>>(level, parent, cu_seqlens, B, T, n_levels, rank, pvec);
    count_launch();
    const int half = d_model / 2;
    const int gx = (half + 127) / 128;
    int tokens_per_cta = 32;
    while ((long long)gx * ((T + tokens_per_cta - 1) / tokens_per_cta) > 65535LL * 4 && tokens_per_cta < (1 << 20)) tokens_per_cta *= 2;
    const dim3 grid(gx, (T + tokens_per_cta - 1) / tokens_per_cta);
    if (grid.y > 65535) return set_error(HDT_ERR_UNSUPPORTED, "hdt_hpe: too many tokens");
    if (dtype == HDT_BF16) k_hpe_eval<true><<<grid, 128, 0, st>>>(level, pvec, T, n_levels, d_model, accumulate, tokens_per_cta, x);
    else k_hpe_eval<false><<<grid, 128, 0, st>>>(level, pvec, T, n_levels, d_model, accumulate, tokens_per_cta, x);
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;
}
