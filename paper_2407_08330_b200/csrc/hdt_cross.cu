// Decoder cross-attention to a level subset of the encoder tokens (paper, paragraph "Results on
// FacetSum (Encoder-Decoder Models)": the decoder attends only to [SEC] anchors, to [SEC] and
// [SENT] anchors, or to all tokens of the encoder output; decoder of the paragraph "Hierarchical
// Encoder and Decoder Stacks").  Within the chosen subset it is plain softmax attention between
// the decoder rows of a document and the chosen encoder rows of the same document.
//
// The chosen rows are never copied.  Every call builds (count, scan, fill: three small kernels,
// 32 CTAs per document, no host wait) one element space for both sides: elements 0 .. Tq-1 are
// the decoder rows (token map = identity, into Q / dO / O), elements Tq .. Tq+ns-1 the chosen
// encoder tokens in order (token map = their index, into K / V); a decoder row's key range is its
// document's slice of the second part, a chosen token's range the document's decoder rows.  The
// attention kernels of the hierarchical path take any (row blocks, per-row range, token map)
// description, so they serve as they are:
//   bf16  the gathering tcgen05 kernels (128-row blocks): forward over the decoder-row blocks;
//         backward once over the decoder-row blocks (dQ) and once over the blocks of chosen
//         tokens (dK, dV); their epilogues round to bf16 and write each element's rows at its token in
//         the caller's tensors (no fp32 buffers, no convert pass);
//   fp32  the SIMT kernels (32-row blocks), which write the caller's tensors directly.
// Encoder rows outside the subset get zero dK, dV (cleared first).  Block slots are assigned
// without a scan: document b owns the slots from start / rows_per_block + b on, unused slots stay
// empty (r0 == r1).
#include <cuda_bf16.h>

#include "hdt_internal.cuh"

namespace hdt {

constexpr int XC = 32;      // CTAs (contiguous chunks) per document in the selection kernels

struct CrossLayout {
    size_t cnt, cntc, cu_sel, tokx, rngx, blocks_q, blocks_k, queue, delta, total;
    int nbq, nbk, xr;
    size_t zero_bytes;      // cnt .. tokx is cleared at the start of every call
};

static size_t al256c(size_t v) { return (v + 255) & ~size_t(255); }

// tc: bf16 on the tensor-core kernels (128-row blocks)
static CrossLayout cross_layout(int B, int T, int Tq, int H, int D, bool tc, int bwd) {
    CrossLayout L{};
    L.xr = tc ? 128 : 32;
    L.nbq = Tq / L.xr + B + 1;
    L.nbk = T / L.xr + B + 1;
    const size_t n = (size_t)Tq + T;
    size_t o = 0;
    L.cnt = o; o += al256c(sizeof(int) * (size_t)(B + 1));
    L.cntc = o; o += al256c(sizeof(int) * (size_t)(B + 1) * XC);
    L.cu_sel = o; o += al256c(sizeof(int) * (size_t)(B + 2));
    L.blocks_q = o; o += al256c(sizeof(int) * 5 * (size_t)L.nbq);
    L.blocks_k = o; o += al256c(sizeof(int) * 5 * (size_t)L.nbk);
    L.tokx = o; o += al256c(sizeof(int) * max(n, (size_t)1));
    L.zero_bytes = o;
    L.rngx = o; o += al256c(sizeof(int) * 2 * max(n, (size_t)1));
    L.queue = o; o += al256c(sizeof(int) * (size_t)max(L.nbq, L.nbk));
    L.delta = o; if (bwd) o += al256c(sizeof(float) * (size_t)H * max(Tq, 1));
    L.total = o + 256;
    return L;
}

__device__ __forceinline__ int chosen(const int8_t *level, int i, int level_mask) {
    const int lv = level[i];
    return (lv >= 0 && lv < 31 && ((level_mask >> lv) & 1)) ? 1 : 0;
}

// cnt[b] = chosen tokens of document b; cntc[b][y] = those in its y-th chunk (XC equal chunks)
__global__ void k_cross_count(const int8_t *__restrict__ level, const int32_t *__restrict__ cu_k, int level_mask,
                              int *cnt, int *cntc) {
    __shared__ int s_c;
    const int b = blockIdx.x, y = blockIdx.y;
    const int k0 = cu_k[b], k1 = cu_k[b + 1], cs = (k1 - k0 + XC - 1) / XC;
    const int c0 = k0 + y * cs, c1 = min(k1, c0 + cs);
    if (threadIdx.x == 0) s_c = 0;
    __syncthreads();
    int c = 0;
    for (int i = c0 + threadIdx.x; i < c1; i += blockDim.x) c += chosen(level, i, level_mask);
    for (int o = 16; o; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(&s_c, c);
    __syncthreads();
    if (threadIdx.x == 0) {
        cntc[b * XC + y] = s_c;
        if (s_c) atomicAdd(&cnt[b], s_c);
    }
}

// cu_sel = exclusive scan of cnt (one CTA); queue = identity
__global__ void __launch_bounds__(1024) k_cross_scan(const int *__restrict__ cnt, int B, int *cu_sel, int *queue, int nq) {
    __shared__ int s_w[32];
    __shared__ int s_carry;
    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    if (t == 0) s_carry = 0;
    __syncthreads();
    for (int base = 0; base < B; base += 1024) {
        const int b = base + t;
        const int c = (b < B) ? cnt[b] : 0;
        int v = c;
        for (int o = 1; o < 32; o <<= 1) { const int x = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += x; }
        if (lane == 31) s_w[w] = v;
        __syncthreads();
        if (w == 0) {
            int x = s_w[lane];
            for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, x, o); if (lane >= o) x += y; }
            s_w[lane] = x;
        }
        __syncthreads();
        if (b < B) cu_sel[b] = s_carry + (w ? s_w[w - 1] : 0) + v - c;
        __syncthreads();
        if (t == 0) s_carry += s_w[31];
        __syncthreads();
    }
    if (t == 0) cu_sel[B] = s_carry;
    for (int i = t; i < nq; i += 1024) queue[i] = i;
}

// Chunk y of document b: its part of the ordered list of chosen tokens (elements KO + position, with
// their row ranges) and its share of the document's decoder rows (elements = row numbers: token
// map, key range) and of the block records of both sides.  xr = rows per block.
__global__ void __launch_bounds__(256) k_cross_fill(const int8_t *__restrict__ level, const int32_t *__restrict__ cu_k,
                                                    const int32_t *__restrict__ cu_q, int level_mask,
                                                    const int *__restrict__ cu_sel, const int *__restrict__ cntc, int KO,
                                                    int xr, int *tokx, int *rngx, int *blocks_q, int *blocks_k) {
    __shared__ int s_w[8];
    __shared__ int s_carry;
    const int b = blockIdx.x, y = blockIdx.y, t = threadIdx.x, lane = t & 31, w = t >> 5;
    const int k0 = cu_k[b], k1 = cu_k[b + 1], q0 = cu_q[b], q1 = cu_q[b + 1], s0 = cu_sel[b], s1 = cu_sel[b + 1];
    const int cs = (k1 - k0 + XC - 1) / XC, c0 = k0 + y * cs, c1 = min(k1, c0 + cs);
    if (w == 0) {       // chosen tokens of the chunks before this one
        int v = (lane < y) ? cntc[b * XC + lane] : 0;       // XC == 32: one lane per chunk
        for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) s_carry = v;
    }
    __syncthreads();
    for (int base = c0; base < c1; base += 256) {
        const int i = base + t;
        const int f = (i < c1) ? chosen(level, i, level_mask) : 0;
        int v = f;
        for (int o = 1; o < 32; o <<= 1) { const int x = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += x; }
        if (lane == 31) s_w[w] = v;
        __syncthreads();
        int before = s_carry;
        for (int j = 0; j < w; ++j) before += s_w[j];
        if (f) {
            const int e = KO + s0 + before + v - 1;
            tokx[e] = i;
            rngx[2 * e] = q0;
            rngx[2 * e + 1] = q1;
        }
        __syncthreads();
        if (t == 0) { int tot = 0; for (int j = 0; j < 8; ++j) tot += s_w[j]; s_carry += tot; }
        __syncthreads();
    }
    // decoder rows and block records: spread over the document's chunks
    const int nt = XC * 256, gt = y * 256 + t;
    for (int r = q0 + gt; r < q1; r += nt) { tokx[r] = r; rngx[2 * r] = KO + s0; rngx[2 * r + 1] = KO + s1; }
    const int live = (s1 > s0 && q1 > q0) ? 0 : HDT_BLK_EMPTY;
    const int slot_q = q0 / xr + b, nbq = (q1 - q0 + xr - 1) / xr;
    for (int j = gt; j < nbq; j += nt) {
        int *rec = blocks_q + 5 * (size_t)(slot_q + j);
        rec[0] = q0 + j * xr; rec[1] = min(q1, q0 + (j + 1) * xr); rec[2] = KO + s0; rec[3] = KO + s1; rec[4] = live;
    }
    const int slot_k = s0 / xr + b, nbk = (s1 - s0 + xr - 1) / xr;
    for (int j = gt; j < nbk; j += nt) {
        int *rec = blocks_k + 5 * (size_t)(slot_k + j);
        rec[0] = KO + s0 + j * xr; rec[1] = KO + min(s1, s0 + (j + 1) * xr); rec[2] = q0; rec[3] = q1; rec[4] = live;
    }
}

static int cross_build(const CrossLayout &L, char *ws, const int8_t *level, const int32_t *cu_k, const int32_t *cu_q,
                       int B, int Tq, int level_mask, cudaStream_t st) {
    // the token map is cleared as a whole: tiles of the gathering kernels reach past the elements
    // in use, and element 0 is a valid row of every tensor
    HDT_CUDA_CHECK(cudaMemsetAsync(ws, 0, L.zero_bytes, st));
    if (B > 0) {
        static_assert(XC == 32, "k_cross_fill sums the chunk counts with one lane per chunk");
        k_cross_count<<<dim3(B, XC), 256, 0, st>>>(level, cu_k, level_mask, (int *)(ws + L.cnt), (int *)(ws + L.cntc));
        k_cross_scan<<<1, 1024, 0, st>>>((const int *)(ws + L.cnt), B, (int *)(ws + L.cu_sel), (int *)(ws + L.queue),
                                         max(L.nbq, L.nbk));
        k_cross_fill<<<dim3(B, XC), 256, 0, st>>>(level, cu_k, cu_q, level_mask, (const int *)(ws + L.cu_sel),
                                                  (const int *)(ws + L.cntc), Tq, L.xr, (int *)(ws + L.tokx),
                                                  (int *)(ws + L.rngx), (int *)(ws + L.blocks_q), (int *)(ws + L.blocks_k));
        count_launch(3);
    }
    HDT_CUDA_CHECK(cudaGetLastError());
    return HDT_OK;
}

static int cross_check(const void *level, const void *cu_k, const void *cu_q, int B, int T, int Tq, int H, int D,
                       int dtype, int level_mask, const void *ws, size_t ws_bytes, size_t need, const char *who) {
    if (B < 0 || T < 0 || Tq < 0 || H < 1) return set_error(HDT_ERR_INVALID_ARG, "%s: negative size or no head", who);
    if (D != 64 && D != 128) return set_error(HDT_ERR_UNSUPPORTED, "%s: head_dim %d not supported (64 or 128)", who, D);
    if (dtype != HDT_F32 && dtype != HDT_BF16) return set_error(HDT_ERR_UNSUPPORTED, "%s: unknown dtype %d", who, dtype);
    if (level_mask < 0) return set_error(HDT_ERR_INVALID_ARG, "%s: level_mask must be a set of level bits 0..30", who);
    if (!cu_k || !cu_q || (T > 0 && !level)) return set_error(HDT_ERR_INVALID_ARG, "%s: null structure pointer", who);
    if (!ws || ws_bytes < need) return set_error(HDT_ERR_WORKSPACE, "%s: workspace %zu < required %zu", who, ws_bytes, need);
    if ((uintptr_t)ws & 255) return set_error(HDT_ERR_INVALID_ARG, "%s: workspace must be 256-byte aligned", who);
    return HDT_OK;
}

}  // namespace hdt

using namespace hdt;

static bool cross_tc(int dtype) { return dtype == HDT_BF16 && !g_force_simt; }

extern "C" size_t hdt_cross_workspace_bytes(int32_t batch, int32_t total_tokens, int32_t total_q, int32_t heads,
                                            int32_t head_dim, int32_t dtype, int32_t bwd) {
    if (batch < 0 || total_tokens < 0 || total_q < 0 || heads < 1 || (head_dim != 64 && head_dim != 128)) return 0;
    // sized for the tensor-core path whenever the dtype allows it (the larger of the two layouts)
    return cross_layout(batch, total_tokens, total_q, heads, head_dim, dtype == HDT_BF16, bwd).total;
}

extern "C" int hdt_cross_attn_fwd(const int8_t *level, const int32_t *cu_seqlens_k, const int32_t *cu_seqlens_q,
                                  int32_t batch, int32_t total_tokens, int32_t total_q, int32_t level_mask,
                                  const void *q, const void *k, const void *v, void *o, float *lse, int32_t heads,
                                  int32_t head_dim, int32_t dtype, float softmax_scale, void *workspace,
                                  size_t workspace_bytes, void *stream) {
    const size_t need = hdt_cross_workspace_bytes(batch, total_tokens, total_q, heads, head_dim, dtype, 0);
    int rc = cross_check(level, cu_seqlens_k, cu_seqlens_q, batch, total_tokens, total_q, heads, head_dim, dtype,
                         level_mask, workspace, workspace_bytes, need, "hdt_cross_attn_fwd");
    if (rc) return rc;
    if (total_q == 0) return HDT_OK;
    if (!q || !o || !lse || (total_tokens > 0 && (!k || !v)))
        return set_error(HDT_ERR_INVALID_ARG, "hdt_cross_attn_fwd: null tensor pointer");
    const bool tc = cross_tc(dtype);
    const CrossLayout L = cross_layout(batch, total_tokens, total_q, heads, head_dim, tc, 0);
    cudaStream_t st = (cudaStream_t)stream;
    char *ws = (char *)workspace;
    rc = cross_build(L, ws, level, cu_seqlens_k, cu_seqlens_q, batch, total_q, level_mask, st);
    if (rc) return rc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
    FwdStageArgs a{};
    a.n = total_q + total_tokens; a.nb = L.nbq; a.H = heads; a.T = total_q;
    a.tok = (const int *)(ws + L.tokx);
    a.tok_rows = a.tok;
    a.rng = (const int *)(ws + L.rngx); a.blocks = (const int *)(ws + L.blocks_q);
    a.queue = (const int *)(ws + L.queue); a.queue_split = a.queue;
    a.q = q; a.k = k; a.v = v; a.o = o; a.lse = lse;
    a.scale_log2 = scale * 1.4426950408889634f;
    a.status = device_status_ptr();
    a.block_rows = L.xr; a.dirs = 7;
    if (!tc) return launch_fwd_simt(a, head_dim, dtype, st);
    a.final_merge = 2;       // the kernel's epilogue writes the bf16 rows and the LSE of the decoder rows itself
    return launch_fwd_tc_upper(a, head_dim, st);
}

extern "C" int hdt_cross_attn_bwd(const int8_t *level, const int32_t *cu_seqlens_k, const int32_t *cu_seqlens_q,
                                  int32_t batch, int32_t total_tokens, int32_t total_q, int32_t level_mask,
                                  const void *q, const void *k, const void *v, const void *o, const float *lse,
                                  const void *d_o, void *dq, void *dk, void *dv, int32_t heads, int32_t head_dim,
                                  int32_t dtype, float softmax_scale, void *workspace, size_t workspace_bytes,
                                  void *stream) {
    const size_t need = hdt_cross_workspace_bytes(batch, total_tokens, total_q, heads, head_dim, dtype, 1);
    int rc = cross_check(level, cu_seqlens_k, cu_seqlens_q, batch, total_tokens, total_q, heads, head_dim, dtype,
                         level_mask, workspace, workspace_bytes, need, "hdt_cross_attn_bwd");
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t esz = dtype == HDT_BF16 ? 2 : 4;
    if (total_tokens > 0) {
        if (!dk || !dv) return set_error(HDT_ERR_INVALID_ARG, "hdt_cross_attn_bwd: null tensor pointer");
        // encoder rows outside the subset (and of documents without decoder rows) get zero gradients
        HDT_CUDA_CHECK(cudaMemsetAsync(dk, 0, (size_t)total_tokens * heads * head_dim * esz, st));
        HDT_CUDA_CHECK(cudaMemsetAsync(dv, 0, (size_t)total_tokens * heads * head_dim * esz, st));
    }
    if (total_q == 0) return HDT_OK;
    if (!q || !o || !lse || !d_o || !dq || (total_tokens > 0 && (!k || !v)))
        return set_error(HDT_ERR_INVALID_ARG, "hdt_cross_attn_bwd: null tensor pointer");
    const bool tc = cross_tc(dtype);
    const CrossLayout L = cross_layout(batch, total_tokens, total_q, heads, head_dim, tc, 1);
    char *ws = (char *)workspace;
    rc = cross_build(L, ws, level, cu_seqlens_k, cu_seqlens_q, batch, total_q, level_mask, st);
    if (rc) return rc;
    float *delta = (float *)(ws + L.delta);
    rc = launch_delta(o, d_o, delta, total_q, heads, head_dim, dtype, st);
    if (rc) return rc;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
    BwdStageArgs a{};
    a.n = total_q + total_tokens; a.H = heads; a.T = total_q;
    a.tok = (const int *)(ws + L.tokx); a.tok_rows = a.tok;
    a.rng = (const int *)(ws + L.rngx);
    a.queue = (const int *)(ws + L.queue); a.queue_split = a.queue;
    a.q = q; a.k = k; a.v = v; a.d_o = d_o; a.lse = lse; a.delta = delta;
    a.scale = scale; a.scale_log2 = scale * 1.4426950408889634f;
    a.dq = dq; a.dk = dk; a.dv = dv;
    a.status = device_status_ptr();
    a.block_rows = L.xr; a.dirs = 7;
    a.gather_end_q = total_q;                       // Q, dO have total_q rows
    a.gather_end_k = total_q + total_tokens;
    BwdStageArgs aq = a, ak = a;
    aq.nb = L.nbq; aq.phases = 1; aq.blocks = (const int *)(ws + L.blocks_q);   // decoder rows as queries: dQ
    ak.nb = L.nbk; ak.phases = 2; ak.blocks = (const int *)(ws + L.blocks_k);   // chosen tokens as keys: dK, dV
    if (!tc) {
        rc = launch_bwd_simt(aq, head_dim, dtype, st);
        if (rc) return rc;
        return launch_bwd_simt(ak, head_dim, dtype, st);
    }
    // the epilogues write bf16 rows at the element's token: dq from the first launch (decoder rows, token =
    // row), dk and dv from the second (chosen tokens, token = their encoder row)
    aq.final_merge = 2; ak.final_merge = 2;
    rc = launch_bwd_tc_upper(aq, head_dim, st);
    if (rc) return rc;
    return launch_bwd_tc_upper(ak, head_dim, st);
}
