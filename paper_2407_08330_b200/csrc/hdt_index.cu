// Device-side index builder: (level, parent, cu_seqlens) -> staged family ranges, row blocks,
// work queues.  Integer work only; every array must equal the sequential definition bit for bit.
//
// Per stage (array of n elements in document order):
//   count     cnt[p] = children of p; nlc[p] = children of p that have children
//   ranges    a node whose children are all childless heads a family; head and children get
//             their key range; children of heads (and PAD) are removed for the next stage
//   scan      exclusive prefix sum of the keep flags -> position in the next stage's array
//   compact   tok / par / sequence offsets of the next stage
//   walk      greedy packing of row blocks per sequence (one CTA per sequence, list in smem)
//   blocks    per block key span, flags, cost
//   queue     rank sort by cost (longest first)
#include <cstdio>

#include "hdt_internal.cuh"

namespace hdt {

static constexpr int CHUNK = 1024;  // elements per CTA in the element-wise kernels

struct Layout {
    size_t header, cnt, nlc, pre, keep, fpos, blocksum, bstart, seqcount, cost, stage0, stage_stride;
    size_t s_tok, s_par, s_rng, s_up, s_scu, s_blocks, s_queue, s_queue2;  // offsets inside a stage
    size_t total;
    int capnb, nchunk;
};

static size_t al(size_t x) { return (x + 255) & ~size_t(255); }

static Layout make_layout(int B, int T, int bm, int max_stages) {
    Layout L;
    L.capnb = 2 * (T / bm + 1) + 4 * B + 2;
    L.nchunk = (T + CHUNK - 1) / CHUNK + 1;
    size_t o = 0;
    L.header = o; o += al(sizeof(DevHeader));
    L.cnt = o; o += al(sizeof(int) * (size_t)T);
    L.nlc = o; o += al(sizeof(int) * (size_t)T);
    L.pre = o; o += al(sizeof(int) * (size_t)T);
    L.keep = o; o += al((size_t)T);
    L.fpos = o; o += al((size_t)T);
    L.blocksum = o; o += al(sizeof(int) * (size_t)L.nchunk);
    L.bstart = o; o += al(sizeof(int) * (size_t)L.capnb);
    L.seqcount = o; o += al(sizeof(int) * (size_t)(B + 1));
    L.cost = o; o += al(sizeof(long long) * (size_t)L.capnb);
    L.stage0 = o;
    size_t s = 0;
    L.s_tok = s; s += al(sizeof(int) * (size_t)T);
    L.s_par = s; s += al(sizeof(int) * (size_t)T);
    L.s_rng = s; s += al(sizeof(int) * 2 * (size_t)T);
    L.s_up = s; s += al(sizeof(int) * (size_t)T);
    L.s_scu = s; s += al(sizeof(int) * (size_t)(B + 1));
    L.s_blocks = s; s += al(sizeof(int) * 5 * (size_t)L.capnb);
    L.s_queue = s; s += al(sizeof(int) * (size_t)L.capnb);
    L.s_queue2 = s; s += al(sizeof(int) * (size_t)L.capnb);
    L.stage_stride = s;
    L.total = o + s * (size_t)max_stages;
    return L;
}

__device__ __forceinline__ void dev_fail(DevHeader *h, int code, int pos) {
    if (atomicCAS(&h->status, 0, code) == 0) h->err_pos = pos;
}

// ---------------------------------------------------------------------------------------------
// stage 0 set-up: validation of the caller's arrays, global parent indices
// ---------------------------------------------------------------------------------------------
__global__ void k_init(const int8_t *__restrict__ level, const int32_t *__restrict__ parent,
                       const int32_t *__restrict__ cu, int B, int T, int max_level, DevHeader *hdr,
                       int *tok, int *par, int *scu, int *cnt, int *nlc) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i <= B) {
        const int c = cu[i];
        scu[i] = c;
        if (i == 0 && c != 0) dev_fail(hdr, HDT_ERR_BAD_HIERARCHY, 0);
        if (i == B && c != T) dev_fail(hdr, HDT_ERR_BAD_HIERARCHY, B);
        if (i < B && cu[i + 1] < c) dev_fail(hdr, HDT_ERR_BAD_HIERARCHY, i);
        if (c < 0 || c > T) dev_fail(hdr, HDT_ERR_BAD_HIERARCHY, i);
    }
    if (i == 0) hdr->st[0].n = T;
    if (i >= T) return;
    // sequence of token i: last b with cu[b] <= i  (cu clamped so a bad cu cannot fault)
    int lo = 0, hi = B;  // invariant: cu[lo] <= i
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (cu[mid] <= i) lo = mid; else hi = mid;
    }
    const int s0 = min(max(cu[lo], 0), T);
    const int r = i - s0;
    const int l = level[i], p = parent[i];
    int gp = -1;
    bool ok = true;
    if (l < 0) {
        ok = (l == -1 && p == -1);
    } else {
        if (l > max_level) ok = false;
        if (r <= 0) {
            ok = ok && (r == 0 && l == 0 && p == -1);
        } else {
            if (p < 0 || p >= r) ok = false;
            else {
                gp = s0 + p;
                if ((int)level[gp] != l - 1) ok = false;
            }
            if ((int)level[i - 1] < 0) ok = false;  // PAD only as a suffix
        }
    }
    if (!ok) { dev_fail(hdr, HDT_ERR_BAD_HIERARCHY, i); gp = -1; }
    tok[i] = i;
    par[i] = gp;
    cnt[i] = 0;
    nlc[i] = 0;
}

__global__ void k_count(const DevHeader *hdr, int s, const int *__restrict__ par, int *cnt) {
    const int n = hdr->st[s].n;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const int p = par[e];
        if (p >= 0) atomicAdd(&cnt[p], 1);
    }
}

__global__ void k_nlc(const DevHeader *hdr, int s, const int *__restrict__ par,
                      const int *__restrict__ cnt, int *nlc) {
    const int n = hdr->st[s].n;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const int p = par[e];
        if (p >= 0 && cnt[e] > 0) atomicAdd(&nlc[p], 1);
    }
}

// One CTA per CHUNK elements (needed for the per-chunk keep counts).
__global__ void __launch_bounds__(CHUNK)
k_ranges(DevHeader *hdr, int s, const int8_t *__restrict__ level /* stage 0 only */,
         const int *__restrict__ par, const int *__restrict__ cnt, const int *__restrict__ nlc,
         int *rng, uint8_t *keep, uint8_t *fpos, int *blocksum) {
    const int n = hdr->st[s].n;
    const int e = blockIdx.x * CHUNK + threadIdx.x;
    int kp = 0;
    long long deg = 0;
    if (e < n) {
        const bool real = level ? (level[e] >= 0) : true;
        const int p = par[e], c = cnt[e];
        const bool head = real && ((c > 0 && nlc[e] == 0) || (s == 0 && p < 0 && c == 0));
        int lo = 0, hi = 0, fp = 0;
        kp = real ? 1 : 0;
        if (head) {
            lo = (p < 0) ? e : e + 1;
            hi = e + 1 + c;
        } else if (p >= 0) {
            const int cp = cnt[p];
            if (cp > 0 && nlc[p] == 0) {  // child of a head
                if (!(p < e && e <= p + cp)) dev_fail(hdr, HDT_ERR_BAD_HIERARCHY, e);
                lo = p;
                hi = p + 1 + cp;
                fp = min(e - p, 255);
                kp = 0;
            }
        }
        rng[2 * e] = lo;
        rng[2 * e + 1] = hi;
        keep[e] = (uint8_t)kp;
        fpos[e] = (uint8_t)fp;
        deg = hi - lo;
        if (kp && p >= 0) hdr->st[s].has_next = 1;  // same value from every writer
    }
    // CTA reductions: keep count and nnz
    __shared__ int s_k[32];
    __shared__ long long s_d[32];
    int k = kp;
    long long d = deg;
    for (int o = 16; o; o >>= 1) {
        k += __shfl_xor_sync(0xffffffffu, k, o);
        d += __shfl_xor_sync(0xffffffffu, d, o);
    }
    if ((threadIdx.x & 31) == 0) { s_k[threadIdx.x >> 5] = k; s_d[threadIdx.x >> 5] = d; }
    __syncthreads();
    if (threadIdx.x < 32) {
        k = s_k[threadIdx.x];
        d = s_d[threadIdx.x];
        for (int o = 16; o; o >>= 1) {
            k += __shfl_xor_sync(0xffffffffu, k, o);
            d += __shfl_xor_sync(0xffffffffu, d, o);
        }
        if (threadIdx.x == 0) {
            blocksum[blockIdx.x] = k;
            if (d) atomicAdd((unsigned long long *)&hdr->nnz, (unsigned long long)d);
        }
    }
}

// Exclusive scan of keep[] (per-CTA offset = sum of the chunk counts before it), next-stage tok.
__global__ void __launch_bounds__(CHUNK)
k_scan(DevHeader *hdr, int s, int nchunk_cap, const uint8_t *__restrict__ keep,
       const int *__restrict__ blocksum, const int *__restrict__ tok, int *pre, int *up, int *tok2) {
    const int n = hdr->st[s].n;
    const int nchunk = (n + CHUNK - 1) / CHUNK;
    if ((int)blockIdx.x >= nchunk && blockIdx.x != 0) return;
    __shared__ int s_w[32];
    __shared__ int s_off, s_tot;
    // offset of this chunk and grand total
    int part = 0, tot = 0;
    for (int c = threadIdx.x; c < nchunk; c += CHUNK) {
        const int v = blocksum[c];
        tot += v;
        if (c < (int)blockIdx.x) part += v;
    }
    for (int o = 16; o; o >>= 1) {
        part += __shfl_xor_sync(0xffffffffu, part, o);
        tot += __shfl_xor_sync(0xffffffffu, tot, o);
    }
    __shared__ int s_p[32], s_t[32];
    if ((threadIdx.x & 31) == 0) { s_p[threadIdx.x >> 5] = part; s_t[threadIdx.x >> 5] = tot; }
    __syncthreads();
    if (threadIdx.x < 32) {
        part = s_p[threadIdx.x];
        tot = s_t[threadIdx.x];
        for (int o = 16; o; o >>= 1) {
            part += __shfl_xor_sync(0xffffffffu, part, o);
            tot += __shfl_xor_sync(0xffffffffu, tot, o);
        }
        if (threadIdx.x == 0) { s_off = part; s_tot = tot; }
    }
    __syncthreads();
    const int has_next = hdr->st[s].has_next;
    if (blockIdx.x == 0 && threadIdx.x == 0) hdr->st[s + 1].n = has_next ? s_tot : 0;
    const int e = blockIdx.x * CHUNK + threadIdx.x;
    const int kp = (e < n) ? keep[e] : 0;
    // block exclusive scan
    int v = kp;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    if (lane == 31) s_w[w] = v;
    __syncthreads();
    if (w == 0) {
        int x = s_w[lane];
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += t;
        }
        s_w[lane] = x;
    }
    __syncthreads();
    const int excl = s_off + (w ? s_w[w - 1] : 0) + v - kp;
    if (e < n) {
        pre[e] = excl;
        const int u = (kp && has_next) ? excl : -1;
        up[e] = u;
        if (u >= 0) tok2[u] = tok[e];
    }
}

__global__ void k_compact(const DevHeader *hdr, int s, int B, const int *__restrict__ par,
                          const int *__restrict__ up, const int *__restrict__ pre,
                          const int *__restrict__ scu, int *par2, int *scu2, int *cnt, int *nlc) {
    const int n = hdr->st[s].n, n2 = hdr->st[s + 1].n;
    const int gtid = blockIdx.x * blockDim.x + threadIdx.x, gsz = gridDim.x * blockDim.x;
    for (int e = gtid; e < n; e += gsz) {
        const int u = up[e];
        if (u >= 0) {
            const int p = par[e];
            par2[u] = (p >= 0) ? pre[p] : -1;
        }
    }
    for (int e = gtid; e < n2; e += gsz) { cnt[e] = 0; nlc[e] = 0; }
    for (int b = gtid; b <= B; b += gsz) {
        const int x = scu[b];
        scu2[b] = (n2 > 0) ? ((x < n) ? pre[x] : n2) : 0;
    }
}

// Greedy block packing of one sequence.  fpos[e] = distance of e from the head of its family
// (0 for heads and for elements in no family, capped at 255 >= block_m).
__global__ void k_walk(const DevHeader *hdr, int s, int bm, const int *__restrict__ scu,
                       const uint8_t *__restrict__ fpos, int *bstart, int *seqcount, int smem_cap) {
    extern __shared__ uint8_t s_fp[];
    const int n = hdr->st[s].n;
    const int b = blockIdx.x;
    if (s > 0 && n == 0) { if (threadIdx.x == 0) seqcount[b] = 0; return; }
    const int s0 = scu[b], s1 = scu[b + 1], len = s1 - s0;
    // capacity offset of this sequence in bstart: sum over earlier sequences of 2*ceil(len/bm)+2
    __shared__ int s_red[32];
    int off = 0;
    for (int c = threadIdx.x; c < b; c += blockDim.x) off += 2 * ((scu[c + 1] - scu[c] + bm - 1) / bm) + 2;
    for (int o = 16; o; o >>= 1) off += __shfl_xor_sync(0xffffffffu, off, o);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = off;
    __syncthreads();
    if (threadIdx.x < 32) {
        off = (threadIdx.x < (blockDim.x >> 5)) ? s_red[threadIdx.x] : 0;
        for (int o = 16; o; o >>= 1) off += __shfl_xor_sync(0xffffffffu, off, o);
        if (threadIdx.x == 0) s_red[0] = off;
    }
    __syncthreads();
    off = s_red[0];
    const bool in_smem = len <= smem_cap;
    if (in_smem)
        for (int i = threadIdx.x; i < len; i += blockDim.x) s_fp[i] = fpos[s0 + i];
    __syncthreads();
    if (threadIdx.x != 0) return;
    const uint8_t *fp = in_smem ? s_fp : (fpos + s0);
    int pos = 0, cntb = 0;
    while (pos < len) {
        int end = min(pos + bm, len);
        if (end < len) {
            const int f = fp[end];
            if (f >= 1 && f < end - pos) end -= f;  // cut would split a family that starts after pos
        }
        bstart[off + cntb] = s0 + pos;
        ++cntb;
        pos = end;
    }
    seqcount[b] = cntb;
}

// Block records of one sequence: one warp per block.
__global__ void k_blocks(DevHeader *hdr, int s, int bm, int B, const int *__restrict__ scu,
                         const int *__restrict__ bstart, const int *__restrict__ seqcount,
                         const int *__restrict__ rng, const int *__restrict__ up, int *blocks,
                         long long *cost) {
    const int n = hdr->st[s].n;
    const int b = blockIdx.x;
    if (s > 0 && n == 0) return;
    __shared__ int s_red[2][32];
    int off = 0, base = 0;
    for (int c = threadIdx.x; c < b; c += blockDim.x) {
        off += 2 * ((scu[c + 1] - scu[c] + bm - 1) / bm) + 2;
        base += seqcount[c];
    }
    for (int o = 16; o; o >>= 1) {
        off += __shfl_xor_sync(0xffffffffu, off, o);
        base += __shfl_xor_sync(0xffffffffu, base, o);
    }
    if ((threadIdx.x & 31) == 0) { s_red[0][threadIdx.x >> 5] = off; s_red[1][threadIdx.x >> 5] = base; }
    __syncthreads();
    if (threadIdx.x < 32) {
        const bool in = threadIdx.x < (blockDim.x >> 5);
        off = in ? s_red[0][threadIdx.x] : 0;
        base = in ? s_red[1][threadIdx.x] : 0;
        for (int o = 16; o; o >>= 1) {
            off += __shfl_xor_sync(0xffffffffu, off, o);
            base += __shfl_xor_sync(0xffffffffu, base, o);
        }
        if (threadIdx.x == 0) { s_red[0][0] = off; s_red[1][0] = base; }
    }
    __syncthreads();
    off = s_red[0][0];
    base = s_red[1][0];
    const int nb_seq = seqcount[b], s1 = scu[b + 1];
    if (b == B - 1 && threadIdx.x == 0) hdr->st[s].nb = base + nb_seq;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    long long vis = 0;
    for (int i = w; i < nb_seq; i += nw) {
        const int r0 = bstart[off + i];
        const int r1 = (i + 1 < nb_seq) ? bstart[off + i + 1] : s1;
        int a = INT_MAX, bb = INT_MIN, carry = 0;
        for (int e = r0 + lane; e < r1; e += 32) {
            const int lo = rng[2 * e], hi = rng[2 * e + 1];
            if (hi > lo) { a = min(a, lo); bb = max(bb, hi); }
            if (up[e] >= 0) carry = 1;
        }
        for (int o = 16; o; o >>= 1) {
            a = min(a, __shfl_xor_sync(0xffffffffu, a, o));
            bb = max(bb, __shfl_xor_sync(0xffffffffu, bb, o));
            carry |= __shfl_xor_sync(0xffffffffu, carry, o);
        }
        const bool any = bb > a;
        if (!any) { a = r0; bb = r0; }
        int dense = 1;
        for (int e = r0 + lane; e < r1; e += 32)
            if (rng[2 * e] != a || rng[2 * e + 1] != bb) dense = 0;
        for (int o = 16; o; o >>= 1) dense &= __shfl_xor_sync(0xffffffffu, dense, o);
        if (lane == 0) {
            int fl = 0;
            if (a >= r0 && bb <= r1) fl |= HDT_BLK_SELF;
            if (dense && any) fl |= HDT_BLK_DENSE;
            if (carry) fl |= HDT_BLK_CARRY;
            if (!any) fl |= HDT_BLK_EMPTY;
            int *rec = blocks + 5 * (size_t)(base + i);
            rec[0] = r0; rec[1] = r1; rec[2] = a; rec[3] = bb; rec[4] = fl;
            const long long c = (long long)(r1 - r0) * (long long)(bb - a);
            cost[base + i] = c;
            vis += c;
        }
    }
    if (lane == 0 && vis) atomicAdd((unsigned long long *)&hdr->visited, (unsigned long long)vis);
}

// Rank sort: queue[rank] = block id, cost descending, id ascending.  queue_split: the same order
// inside two groups, blocks that are SELF and not EMPTY first (n_fused of them), then the others.
__global__ void k_queue(DevHeader *hdr, int s, const long long *__restrict__ cost,
                        const int *__restrict__ blocks, int *queue, int *queue_split) {
    const int nb = hdr->st[s].nb;
    int mine = 0;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < nb; i += gridDim.x * blockDim.x) {
        const long long ci = cost[i];
        const int fi = blocks[5 * i + 4];
        const int ei = ((fi & HDT_BLK_SELF) && !(fi & HDT_BLK_EMPTY)) ? 1 : 0;
        int rank = 0, rank2 = 0;
        for (int j = 0; j < nb; ++j) {
            const long long cj = cost[j];
            const int fj = blocks[5 * j + 4];
            const int ej = ((fj & HDT_BLK_SELF) && !(fj & HDT_BLK_EMPTY)) ? 1 : 0;
            const int before = (cj > ci) || (cj == ci && j < i);
            rank += before;
            rank2 += (ej > ei) || (ej == ei && before);
        }
        queue[rank] = i;
        queue_split[rank2] = i;
        mine += ei;
    }
    if (mine) atomicAdd(&hdr->st[s].n_fused, mine);
}

}  // namespace hdt

using namespace hdt;

static void norm_params(const hdt_index_params_t *p, int &bm, int &ms) {
    bm = (p && p->block_m) ? p->block_m : 128;
    ms = (p && p->max_stages) ? p->max_stages : 4;
}

extern "C" size_t hdt_index_workspace_bytes(int32_t batch, int32_t total_tokens,
                                            const hdt_index_params_t *params) {
    int bm, ms;
    norm_params(params, bm, ms);
    if (batch < 0 || total_tokens < 0 || bm < 1 || bm > 128 || ms < 1 || ms > HDT_MAX_STAGES) return 0;
    return make_layout(batch, total_tokens, bm, ms).total;
}

extern "C" int hdt_build_index(const int8_t *level, const int32_t *parent, const int32_t *cu_seqlens,
                               int32_t batch, int32_t total_tokens, const hdt_index_params_t *params,
                               void *workspace, size_t workspace_bytes, void *stream, hdt_index_t **out) {
    if (out) *out = nullptr;
    int bm, ms;
    norm_params(params, bm, ms);
    if (!out || !cu_seqlens || !workspace || batch < 0 || total_tokens < 0 ||
        (total_tokens > 0 && (!level || !parent)))
        return set_error(HDT_ERR_INVALID_ARG, "hdt_build_index: null pointer or negative size");
    if (bm < 1 || bm > 128 || ms < 1 || ms > HDT_MAX_STAGES)
        return set_error(HDT_ERR_INVALID_ARG, "hdt_build_index: block_m must be 1..128, max_stages 1..%d",
                         HDT_MAX_STAGES);
    if (((uintptr_t)workspace & 255) != 0)
        return set_error(HDT_ERR_INVALID_ARG, "hdt_build_index: workspace must be 256-byte aligned");
    const int B = batch, T = total_tokens;
    const Layout L = make_layout(B, T, bm, ms);
    if (workspace_bytes < L.total)
        return set_error(HDT_ERR_WORKSPACE, "hdt_build_index: workspace %zu < required %zu", workspace_bytes,
                         L.total);
    cudaStream_t st = (cudaStream_t)stream;
    char *ws = (char *)workspace;
    DevHeader *hdr = (DevHeader *)(ws + L.header);
    int *cnt = (int *)(ws + L.cnt), *nlc = (int *)(ws + L.nlc), *pre = (int *)(ws + L.pre);
    uint8_t *keep = (uint8_t *)(ws + L.keep), *fpos = (uint8_t *)(ws + L.fpos);
    int *blocksum = (int *)(ws + L.blocksum), *bstart = (int *)(ws + L.bstart);
    int *seqcount = (int *)(ws + L.seqcount);
    long long *cost = (long long *)(ws + L.cost);

    hdt_index *ix = new hdt_index();
    ix->batch = B; ix->total_tokens = T; ix->block_m = bm; ix->n_stages = 0;
    ix->workspace = workspace; ix->workspace_bytes = workspace_bytes;
    for (int s = 0; s < ms; ++s) {
        char *base = ws + L.stage0 + L.stage_stride * (size_t)s;
        ix->st[s] = StagePtrs{(int *)(base + L.s_tok), (int *)(base + L.s_par), (int *)(base + L.s_rng),
                              (int *)(base + L.s_up), (int *)(base + L.s_scu), (int *)(base + L.s_blocks),
                              (int *)(base + L.s_queue), (int *)(base + L.s_queue2)};
    }
#define HDT_BUILD_CHECK(expr)                                                          \
    do {                                                                               \
        cudaError_t e_ = (expr);                                                       \
        if (e_ != cudaSuccess) {                                                       \
            delete ix;                                                                 \
            return set_error(HDT_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_)); \
        }                                                                              \
    } while (0)

    {
    ProfScope ps(PROF_INDEX, st);
    HDT_BUILD_CHECK(cudaMemsetAsync(hdr, 0, sizeof(DevHeader), st));
    const int nel = max(T, B + 1);
    const int g_el = (nel + 255) / 256;
    const int g_chunk = max(1, (T + CHUNK - 1) / CHUNK);
    const int g_stride = max(1, min((T + 255) / 256, 148 * 8));
    static const int kSmemCap = 200 * 1024;
    static bool attr_set = false;
    if (!attr_set) {
        HDT_BUILD_CHECK(cudaFuncSetAttribute(k_walk, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemCap));
        attr_set = true;
    }
    k_init<<<g_el, 256, 0, st>>>(level, parent, cu_seqlens, B, T, HDT_MAX_STAGES * 8, hdr, ix->st[0].tok,
                                 ix->st[0].par, ix->st[0].scu, cnt, nlc);
    count_launch();
    for (int s = 0; s < ms; ++s) {
        const StagePtrs &P = ix->st[s];
        // the last possible stage writes its (unused) next-stage arrays into its own up/pre scratch
        const StagePtrs &N = ix->st[(s + 1 < ms) ? s + 1 : s];
        const bool last = (s + 1 == ms);
        k_count<<<g_stride, 256, 0, st>>>(hdr, s, P.par, cnt);
        k_nlc<<<g_stride, 256, 0, st>>>(hdr, s, P.par, cnt, nlc);
        k_ranges<<<g_chunk, CHUNK, 0, st>>>(hdr, s, s == 0 ? level : nullptr, P.par, cnt, nlc, P.rng, keep,
                                            fpos, blocksum);
        // tok2 of the last possible stage is never read: point it at scratch (pre is rewritten first)
        k_scan<<<g_chunk, CHUNK, 0, st>>>(hdr, s, L.nchunk, keep, blocksum, P.tok, pre, P.up,
                                          last ? cnt : N.tok);
        if (!last) {
            k_compact<<<g_stride, 256, 0, st>>>(hdr, s, B, P.par, P.up, pre, P.scu, N.par, N.scu, cnt, nlc);
            count_launch();
        }
        if (B > 0) {
            int maxlen_smem = kSmemCap;  // sequences longer than this walk through global memory
            k_walk<<<B, 256, kSmemCap, st>>>(hdr, s, bm, P.scu, fpos, bstart, seqcount, maxlen_smem);
            k_blocks<<<B, 256, 0, st>>>(hdr, s, bm, B, P.scu, bstart, seqcount, P.rng, P.up, P.blocks, cost);
            k_queue<<<max(1, min(L.capnb / 128 + 1, 148 * 4)), 128, 0, st>>>(hdr, s, cost, P.blocks, P.queue, P.queue_split);
            count_launch(3);
        }
        count_launch(4);
    }
    HDT_BUILD_CHECK(cudaGetLastError());
    }
    DevHeader h;
    HDT_BUILD_CHECK(cudaMemcpyAsync(&h, hdr, sizeof(DevHeader), cudaMemcpyDeviceToHost, st));
    HDT_BUILD_CHECK(cudaStreamSynchronize(st));
#undef HDT_BUILD_CHECK
    if (h.status != 0) {
        delete ix;
        return set_error(h.status, "hdt_build_index: structure arrays violate a precondition near element %d",
                         h.err_pos);
    }
    int ns = 1;
    while (ns < ms && h.st[ns].n > 0) ++ns;
    if (h.st[ns - 1].has_next && ns == ms) {
        delete ix;
        return set_error(HDT_ERR_BAD_HIERARCHY,
                         "hdt_build_index: hierarchy needs more than max_stages = %d stages", ms);
    }
    // a last stage that found "has_next" without one being built cannot happen below ms
    ix->n_stages = ns;
    ix->nnz = h.nnz;
    ix->visited = h.visited;
    for (int s = 0; s <= HDT_MAX_STAGES; ++s) ix->desc[s] = h.st[s];
    *out = ix;
    return HDT_OK;
}

extern "C" int hdt_index_info(const hdt_index_t *ix, int32_t *n_stages, int64_t *nnz, int64_t *visited) {
    if (!ix) return set_error(HDT_ERR_INVALID_ARG, "hdt_index_info: null index");
    if (n_stages) *n_stages = ix->n_stages;
    if (nnz) *nnz = ix->nnz;
    if (visited) *visited = ix->visited;
    return HDT_OK;
}

extern "C" int hdt_index_export(const hdt_index_t *ix, int32_t stage, hdt_stage_view_t *v) {
    if (!ix || !v) return set_error(HDT_ERR_INVALID_ARG, "hdt_index_export: null argument");
    if (stage < 0 || stage >= ix->n_stages)
        return set_error(HDT_ERR_INVALID_ARG, "hdt_index_export: stage %d outside [0,%d)", stage, ix->n_stages);
    const StagePtrs &P = ix->st[stage];
    v->n = ix->desc[stage].n;
    v->n_blocks = ix->desc[stage].nb;
    v->tok = P.tok; v->par = P.par; v->rng = P.rng; v->up = P.up; v->scu = P.scu;
    v->blocks = P.blocks; v->queue = P.queue;
    v->queue_split = P.queue_split;
    v->n_fused = ix->desc[stage].n_fused;
    return HDT_OK;
}

extern "C" int hdt_index_destroy(hdt_index_t *ix) {
    delete ix;
    return HDT_OK;
}
