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
#include <cstring>
#include <atomic>
#include <mutex>
#include <vector>

#include "hdt_internal.cuh"

namespace hdt {

static constexpr int CHUNK = 1024;  // elements per CTA in the element-wise kernels

struct Layout {
    size_t header, cnt, nlc, pre, keep, fpos, blocksum, bstart, seqcount, cost, stage0, stage_stride;
    size_t fpos2, bstart2, seqcount2, cost2;   // second set for the upper stages, built beside stage 0's blocks
    size_t rank;                               // per token: its number among its siblings (written where its family is found)
    size_t s_tok, s_par, s_rng, s_up, s_scu, s_blocks, s_queue, s_queue2;  // offsets inside a stage
    size_t total;
    int capnb, nchunk;
};

static size_t al(size_t x) { return (x + 255) & ~size_t(255); }

static Layout make_layout(int B, int T, int bm, int max_stages) {   // bm: the smaller of the two block sizes
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
    L.fpos2 = o; o += al((size_t)T);
    L.bstart2 = o; o += al(sizeof(int) * (size_t)L.capnb);
    L.seqcount2 = o; o += al(sizeof(int) * (size_t)(B + 1));
    L.cost2 = o; o += al(sizeof(long long) * (size_t)L.capnb);
    L.rank = o; o += al(sizeof(int) * (size_t)T);
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
    // cnt and nlc were zeroed with the header.  nlc[x] = children of x that have children: the first
    // child to register with its parent reports that parent to the grandparent, once per parent
    // (no second pass over the elements after the counts are complete).
    if (gp >= 0 && atomicAdd(&cnt[gp], 1) == 0) {
        const int pg = parent[gp];
        if (pg >= 0 && pg < gp - s0) atomicAdd(&nlc[s0 + pg], 1);   // (gp's own thread reports a bad entry)
    }
}

// One CTA per CHUNK elements (needed for the per-chunk keep counts).
// Keys of row e with range [lo, hi) that the direction bits keep.  A row whose range starts at or
// after itself is the head of its family (the keys after it are its children); otherwise lo is
// the row's parent and the remaining keys are its siblings.  dirs: 1 = child -> parent,
// 2 = sibling <-> sibling, 4 = parent -> child; the diagonal always stays.
__device__ __forceinline__ int row_pairs(int e, int lo, int hi, int dirs) {
    if (hi <= lo) return 0;
    if (lo >= e) return (lo == e ? 1 : 0) + ((dirs & 4) ? hi - e - 1 : 0);
    return 1 + ((dirs & 1) ? 1 : 0) + ((dirs & 2) ? hi - lo - 2 : 0);
}

__global__ void __launch_bounds__(CHUNK)
k_ranges(DevHeader *hdr, int s, const int8_t *__restrict__ level /* stage 0 only */,
         const int *__restrict__ par, const int *__restrict__ cnt, const int *__restrict__ nlc,
         int *rng, uint8_t *keep, uint8_t *fpos, int *blocksum, int dirs, const int *__restrict__ tok /* nullptr: identity */,
         int *rank) {
    pdl_launch_dependents();      // the kernel queued behind this one may be scheduled now; it waits likewise
    pdl_wait();                   // the kernel before this one has completed
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
                rank[tok ? tok[e] : e] = e - p;     // the token's number among its siblings (hierarchical positions)
            }
        }
        rng[2 * e] = lo;
        rng[2 * e + 1] = hi;
        keep[e] = (uint8_t)kp;
        fpos[e] = (uint8_t)fp;
        deg = row_pairs(e, lo, hi, dirs);
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
       const int *__restrict__ blocksum, const int *__restrict__ tok, int *pre, int *up, int *tok2, int *cnt_clear,
       int *nlc_clear) {
    pdl_launch_dependents();      // the kernel queued behind this one may be scheduled now; it waits likewise
    pdl_wait();                   // the kernel before this one has completed
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
        // (this stage's counts are dead: cleared here where k_compact goes on to count the next stage's children)
        if (cnt_clear != nullptr) { cnt_clear[e] = 0; nlc_clear[e] = 0; }
    }
}

// count_next: cnt and nlc were cleared by k_scan; the next stage's child counts (and nlc, as in k_init) are taken
// here, where its parent indices are formed, instead of in a kernel of their own.
__global__ void k_compact(const DevHeader *hdr, int s, int B, const int *__restrict__ par,
                          const int *__restrict__ up, const int *__restrict__ pre,
                          const int *__restrict__ scu, int *par2, int *scu2, int *cnt, int *nlc, int count_next) {
    pdl_launch_dependents();      // the kernel queued behind this one may be scheduled now; it waits likewise
    pdl_wait();                   // the kernel before this one has completed
    const int n = hdr->st[s].n, n2 = hdr->st[s + 1].n;
    const int gtid = blockIdx.x * blockDim.x + threadIdx.x, gsz = gridDim.x * blockDim.x;
    for (int e = gtid; e < n; e += gsz) {
        const int u = up[e];
        if (u >= 0) {
            const int p = par[e];
            const int q = (p >= 0) ? pre[p] : -1;
            par2[u] = q;
            if (count_next && n2 > 0 && q >= 0 && atomicAdd(&cnt[q], 1) == 0) {      // (a kept element's ancestors are kept)
                const int pp = par[p];
                if (pp >= 0) atomicAdd(&nlc[pre[pp]], 1);
            }
        }
    }
    if (!count_next)
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
    pdl_launch_dependents();      // the kernel queued behind this one may be scheduled now; it waits likewise
    pdl_wait();                   // the kernel before this one has completed
    extern __shared__ __align__(16) uint8_t s_fp[];
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
    // stage fpos[a0 .. s1) from the 16-byte boundary a0 <= s0 with vector loads
    const int a0 = s0 & ~15, skew = s0 - a0;
    const bool in_smem = len + 32 <= smem_cap;
    if (in_smem) {
        const uint4 *src = reinterpret_cast<const uint4 *>(fpos + a0);
        uint4 *dst = reinterpret_cast<uint4 *>(s_fp);
        const int nv = (skew + len + 15) >> 4;   // the workspace array is padded to 256 bytes: no overrun
        for (int i = threadIdx.x; i < nv; i += blockDim.x) dst[i] = src[i];
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    const uint8_t *fp = in_smem ? (s_fp + skew) : (fpos + s0);
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
    pdl_launch_dependents();      // the kernel queued behind this one may be scheduled now; it waits likewise
    pdl_wait();                   // the kernel before this one has completed
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
    if (b == B - 1 && threadIdx.x == 0 && blockIdx.y == 0) hdr->st[s].nb = base + nb_seq;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = blockDim.x >> 5;
    long long vis = 0;
    for (int i = blockIdx.y * nw + w; i < nb_seq; i += nw * gridDim.y) {   // grid.y CTAs share a sequence
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
// One warp per block: its lanes share the scan over all blocks and add up their counts.
__global__ void __launch_bounds__(256)
k_queue(DevHeader *hdr, int s, const long long *__restrict__ cost, const int *__restrict__ blocks, int *queue,
        int *queue_split) {
    pdl_launch_dependents();      // the kernel queued behind this one may be scheduled now; it waits likewise
    pdl_wait();                   // the kernel before this one has completed
    const int nb = hdr->st[s].nb;
    const int lane = threadIdx.x & 31;
    const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nw = (gridDim.x * blockDim.x) >> 5;
    int mine = 0, mine_empty = 0;
    for (int i = gw; i < nb; i += nw) {
        const long long ci = cost[i];
        const int fi = blocks[5 * i + 4];
        const int ei = ((fi & HDT_BLK_SELF) && !(fi & HDT_BLK_EMPTY)) ? 1 : 0;
        int rank = 0, rank2 = 0;
        for (int j = lane; j < nb; j += 32) {
            const long long cj = cost[j];
            const int fj = blocks[5 * j + 4];
            const int ej = ((fj & HDT_BLK_SELF) && !(fj & HDT_BLK_EMPTY)) ? 1 : 0;
            const int before = (cj > ci) || (cj == ci && j < i);
            rank += before;
            rank2 += (ej > ei) || (ej == ei && before);
        }
        for (int o = 16; o; o >>= 1) {
            rank += __shfl_xor_sync(0xffffffffu, rank, o);
            rank2 += __shfl_xor_sync(0xffffffffu, rank2, o);
        }
        if (lane == 0) {
            queue[rank] = i;
            queue_split[rank2] = i;
            mine += ei;
            mine_empty += (fi & HDT_BLK_EMPTY) ? 1 : 0;
        }
    }
    if (lane == 0 && mine) atomicAdd(&hdr->st[s].n_fused, mine);
    if (lane == 0 && mine_empty) atomicAdd(&hdr->st[s].n_empty, mine_empty);
}

// ---------------------------------------------------------------------------------------------
// All stages above 0 in one CTA.  Their arrays are a few percent of the tokens, so a single CTA
// with block-wide barriers between the steps replaces eight launches per stage.
// ---------------------------------------------------------------------------------------------
struct UpperArgs {
    StagePtrs st[HDT_MAX_STAGES];
    int max_stages, B, bm, dirs;
    int *cnt, *nlc, *pre, *bstart, *seqcount, *rank;
    uint8_t *keep, *fpos;
    long long *cost;
};

static constexpr int UT = 1024;      // threads of the fused kernel
static constexpr int UMAXB = 1024;   // sequences it handles (per-sequence offsets live in shared memory)
static constexpr int UCAP = 4096;    // elements of a stage whose scratch fits in shared memory
static constexpr int USB = 2048;     // block slots of a stage whose block starts, costs and flags stay in shared memory
static constexpr int USMEM = UCAP * (8 * 4 + 2) + USB * (4 + 8 + 1);   // bytes of that scratch

__global__ void __launch_bounds__(UT) k_upper_stages(DevHeader *hdr, const UpperArgs u) {
    // Stages of at most UCAP elements keep their per-element scratch (tokens, parents, child counts,
    // keep flags, prefix sums, ranges, next-stage indices) in shared memory, and with at most USB
    // block slots the block starts, costs and flags too: a dozen barrier-separated steps per stage
    // would otherwise each pay a round trip to global memory (after the loads at a stage's start
    // such a stage only writes to it).
    extern __shared__ __align__(16) int s_dyn[];
    int *s_par = s_dyn, *s_cnt = s_par + UCAP, *s_nlc = s_cnt + UCAP, *s_pre = s_nlc + UCAP, *s_up = s_pre + UCAP;
    int *s_rng = s_up + UCAP;                                   // 2 * UCAP
    int *s_tok = s_rng + 2 * UCAP;
    long long *s_cst = reinterpret_cast<long long *>(s_tok + UCAP);   // (8-byte aligned: the arrays before it are multiples of 16 KB)
    int *s_bst = reinterpret_cast<int *>(s_cst + USB);
    uint8_t *s_keep = reinterpret_cast<uint8_t *>(s_bst + USB), *s_fpos = s_keep + UCAP, *s_bfl = s_fpos + UCAP;
    __shared__ int s_off[UMAXB], s_base[UMAXB + 1], s_nbs[UMAXB], s_scu[UMAXB + 1];   // per sequence: block slots, first block, block count, offsets
    __shared__ int s_w[32];
    __shared__ int s_carry, s_flag, s_cap;
    __shared__ long long s_ll[32];
    const int t = threadIdx.x, lane = t & 31, w = t >> 5;
    const int B = u.B, bm = u.bm;
    int n = hdr->st[1].n;                // (stage 0's kernels wrote it; the later ones are computed here)
    for (int s = 1; s < u.max_stages; ++s) {
        if (n == 0) break;
        const StagePtrs P = u.st[s];
        const bool last = (s + 1 == u.max_stages);
        const StagePtrs N = u.st[last ? s : s + 1];
        const bool small = n <= UCAP;
        int *cnt = small ? s_cnt : u.cnt, *nlc = small ? s_nlc : u.nlc, *pre = small ? s_pre : u.pre;
        uint8_t *keep = small ? s_keep : u.keep, *fpos = small ? s_fpos : u.fpos;
        const int *par = small ? s_par : P.par, *tokr = small ? s_tok : P.tok;
        const int *rngr = small ? s_rng : P.rng, *upr = small ? s_up : P.up;    // read-back of this stage's results
        for (int b = t; b <= B; b += UT) s_scu[b] = P.scu[b];
        if (small)
            for (int e = t; e < n; e += UT) { s_par[e] = P.par[e]; s_tok[e] = P.tok[e]; s_cnt[e] = 0; s_nlc[e] = 0; }
        __syncthreads();
        // children counts (cnt, nlc are zero for [0, n))
        for (int e = t; e < n; e += UT) { const int p = par[e]; if (p >= 0) atomicAdd(&cnt[p], 1); }
        if (t == 0) { s_flag = 0; s_carry = 0; }
        __syncthreads();
        for (int e = t; e < n; e += UT) { const int p = par[e]; if (p >= 0 && cnt[e] > 0) atomicAdd(&nlc[p], 1); }
        __syncthreads();
        // ranges, keep flags
        long long deg = 0;
        for (int e = t; e < n; e += UT) {
            const int p = par[e], c = cnt[e];
            const bool head = (c > 0 && nlc[e] == 0);
            int lo = 0, hi = 0, fp = 0, kp = 1;
            if (head) {
                lo = (p < 0) ? e : e + 1;
                hi = e + 1 + c;
            } else if (p >= 0) {
                const int cp = cnt[p];
                if (cp > 0 && nlc[p] == 0) {
                    if (!(p < e && e <= p + cp)) dev_fail(hdr, HDT_ERR_BAD_HIERARCHY, e);
                    lo = p; hi = p + 1 + cp; fp = min(e - p, 255); kp = 0;
                    u.rank[tokr[e]] = e - p;
                }
            }
            P.rng[2 * e] = lo;
            P.rng[2 * e + 1] = hi;
            if (small) { s_rng[2 * e] = lo; s_rng[2 * e + 1] = hi; }
            keep[e] = (uint8_t)kp;
            fpos[e] = (uint8_t)fp;
            deg += row_pairs(e, lo, hi, u.dirs);
            if (kp && p >= 0) s_flag = 1;
        }
        for (int o = 16; o; o >>= 1) deg += __shfl_xor_sync(0xffffffffu, deg, o);
        if (lane == 0) s_ll[w] = deg;
        __syncthreads();
        if (t == 0) {
            long long d = 0;
            for (int i = 0; i < UT / 32; ++i) d += s_ll[i];
            if (d) atomicAdd((unsigned long long *)&hdr->nnz, (unsigned long long)d);
            hdr->st[s].has_next = s_flag;
        }
        const int has_next = s_flag;
        // exclusive scan of keep[] in chunks of UT
        for (int base = 0; base < n; base += UT) {
            const int e = base + t;
            const int kp = (e < n) ? keep[e] : 0;
            int v = kp;
            for (int o = 1; o < 32; o <<= 1) { const int x = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += x; }
            if (lane == 31) s_w[w] = v;
            __syncthreads();
            if (w == 0) {
                int x = s_w[lane];
                for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, x, o); if (lane >= o) x += y; }
                s_w[lane] = x;
            }
            __syncthreads();
            const int excl = s_carry + (w ? s_w[w - 1] : 0) + v - kp;
            if (e < n) {
                pre[e] = excl;
                const int up = (kp && has_next) ? excl : -1;
                P.up[e] = up;
                if (small) s_up[e] = up;
                if (up >= 0 && !last) N.tok[up] = tokr[e];
            }
            __syncthreads();
            if (t == 0) s_carry += s_w[31];
            __syncthreads();
        }
        const int n2 = has_next ? s_carry : 0;
        if (t == 0) hdr->st[s + 1].n = n2;
        // next stage's parents and sequence offsets; clear cnt / nlc for it
        if (!last) {
            for (int e = t; e < n; e += UT) {
                const int up = upr[e];
                if (up >= 0) { const int p = par[e]; N.par[up] = (p >= 0) ? pre[p] : -1; }
            }
            for (int b = t; b <= B; b += UT) {
                const int x = s_scu[b];
                N.scu[b] = (n2 > 0) ? ((x < n) ? pre[x] : n2) : 0;
            }
        }
        __syncthreads();   // every cnt / nlc / pre read of this stage is done
        if (!small)
            for (int e = t; e < max(n2, 0); e += UT) { u.cnt[e] = 0; u.nlc[e] = 0; }
        // per-sequence capacity offsets, greedy walk (one lane per sequence)
        for (int b = t; b < B; b += UT) {
            int off = 0;
            for (int c = 0; c < b; ++c) off += 2 * ((s_scu[c + 1] - s_scu[c] + bm - 1) / bm) + 2;
            s_off[b] = off;
            if (b == B - 1) s_cap = off + 2 * ((s_scu[b + 1] - s_scu[b] + bm - 1) / bm) + 2;
        }
        __syncthreads();
        const bool few = B > 0 && s_cap <= USB;        // block slots of this stage fit in shared memory
        int *bst = few ? s_bst : u.bstart;
        long long *cst = few ? s_cst : u.cost;
        for (int b = w; b < B; b += UT / 32) {
            if (lane == 0) {
                const int s0 = s_scu[b], len = s_scu[b + 1] - s0, off = s_off[b];
                int pos = 0, cntb = 0;
                while (pos < len) {
                    int end = min(pos + bm, len);
                    if (end < len) {
                        const int f = fpos[s0 + end];
                        if (f >= 1 && f < end - pos) end -= f;
                    }
                    bst[off + cntb] = s0 + pos;
                    ++cntb;
                    pos = end;
                }
                u.seqcount[b] = cntb;
                s_nbs[b] = cntb;
            }
        }
        __syncthreads();
        for (int b = t; b < B; b += UT) {
            int base = 0;
            for (int c = 0; c < b; ++c) base += s_nbs[c];
            s_base[b] = base;
            if (b == B - 1) { hdr->st[s].nb = base + s_nbs[b]; s_base[B] = base + s_nbs[b]; }
        }
        __syncthreads();
        // block records, one warp per block over all sequences (the block's sequence by bisection of s_base)
        long long vis = 0;
        {
            const int nb_all = (B > 0) ? s_base[B] : 0;
            for (int gb = w; gb < nb_all; gb += UT / 32) {
                int lo_b = 0, hi_b = B;
                while (hi_b - lo_b > 1) { const int mid = (lo_b + hi_b) >> 1; if (s_base[mid] <= gb) lo_b = mid; else hi_b = mid; }
                // (the largest b with s_base[b] <= gb always owns blocks: an empty sequence has the base of its successor)
                const int b = lo_b, i = gb - s_base[b];
                const int nb_seq = s_nbs[b], off = s_off[b], base = s_base[b], s1 = s_scu[b + 1];
                const int r0 = bst[off + i];
                const int r1 = (i + 1 < nb_seq) ? bst[off + i + 1] : s1;
                int a = 0x7fffffff, bb = (int)0x80000000, carry = 0;
                for (int e = r0 + lane; e < r1; e += 32) {
                    const int lo = rngr[2 * e], hi = rngr[2 * e + 1];
                    if (hi > lo) { a = min(a, lo); bb = max(bb, hi); }
                    if (upr[e] >= 0) carry = 1;
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
                    if (rngr[2 * e] != a || rngr[2 * e + 1] != bb) dense = 0;
                for (int o = 16; o; o >>= 1) dense &= __shfl_xor_sync(0xffffffffu, dense, o);
                if (lane == 0) {
                    int fl = 0;
                    if (a >= r0 && bb <= r1) fl |= HDT_BLK_SELF;
                    if (dense && any) fl |= HDT_BLK_DENSE;
                    if (carry) fl |= HDT_BLK_CARRY;
                    if (!any) fl |= HDT_BLK_EMPTY;
                    int *rec = P.blocks + 5 * (size_t)(base + i);
                    rec[0] = r0; rec[1] = r1; rec[2] = a; rec[3] = bb; rec[4] = fl;
                    const long long c = (long long)(r1 - r0) * (long long)(bb - a);
                    cst[base + i] = c;
                    if (few) s_bfl[base + i] = (uint8_t)fl;
                    vis += c;
                }
            }
        }
        if (lane == 0 && vis) atomicAdd((unsigned long long *)&hdr->visited, (unsigned long long)vis);
        __syncthreads();
        // queues
        const int nb = (B > 0) ? s_base[B] : 0;
        int mine = 0, mine_empty = 0;
        for (int i = w; i < nb; i += UT / 32) {      // one warp per block, lanes share the scan
            const long long ci = cst[i];
            const int fi = few ? (int)s_bfl[i] : P.blocks[5 * i + 4];
            const int ei = ((fi & HDT_BLK_SELF) && !(fi & HDT_BLK_EMPTY)) ? 1 : 0;
            int rank = 0, rank2 = 0;
            for (int j = lane; j < nb; j += 32) {
                const long long cj = cst[j];
                const int fj = few ? (int)s_bfl[j] : P.blocks[5 * j + 4];
                const int ej = ((fj & HDT_BLK_SELF) && !(fj & HDT_BLK_EMPTY)) ? 1 : 0;
                const int before = (cj > ci) || (cj == ci && j < i);
                rank += before;
                rank2 += (ej > ei) || (ej == ei && before);
            }
            for (int o = 16; o; o >>= 1) {
                rank += __shfl_xor_sync(0xffffffffu, rank, o);
                rank2 += __shfl_xor_sync(0xffffffffu, rank2, o);
            }
            if (lane == 0) {
                P.queue[rank] = i;
                P.queue_split[rank2] = i;
                mine += ei;
                mine_empty += (fi & HDT_BLK_EMPTY) ? 1 : 0;
            }
        }
        if (mine) atomicAdd(&hdr->st[s].n_fused, mine);
        if (mine_empty) atomicAdd(&hdr->st[s].n_empty, mine_empty);
        __syncthreads();   // every read of this stage's scratch is done before the next stage overwrites it
        n = n2;
    }
}

}  // namespace hdt

using namespace hdt;

static int norm_dirs(const hdt_index_params_t *p) { return p ? (~p->mask_off) & 7 : 7; }

static void norm_params(const hdt_index_params_t *p, int &bm, int &ms, int &bmu) {
    bm = (p && p->block_m) ? p->block_m : 128;
    ms = (p && p->max_stages) ? p->max_stages : 4;
    bmu = (p && p->block_m_upper) ? p->block_m_upper : 128;
}

extern "C" size_t hdt_index_workspace_bytes(int32_t batch, int32_t total_tokens,
                                            const hdt_index_params_t *params) {
    int bm, ms, bmu;
    norm_params(params, bm, ms, bmu);
    if (batch < 0 || total_tokens < 0 || bm < 1 || bm > 128 || bmu < 1 || bmu > 128 || ms < 1 || ms > HDT_MAX_STAGES)
        return 0;
    return make_layout(batch, total_tokens, min(bm, bmu), ms).total;
}

// Launch as a programmatic dependent of the kernel before it on the stream (its CTAs are scheduled
// while that kernel ends and wait for it with pdl_wait): the dozen tiny kernels of a build are a
// chain, and most of each link is launch latency.
template <typename... KArgs, typename... Args>
static cudaError_t launch_chain(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = g_no_pdl ? 0 : 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// Pinned landing buffers for index headers: a small pool shared by all host threads (a deferred
// index keeps its buffer until the header has been read).
static const int kUnset = 0x7fffffff;
static std::mutex g_pinned_mu;
// A landing buffer for the header with the event that marks the end of its copy.
struct PinnedSlot { DevHeader *p; cudaEvent_t ev; };
static std::vector<PinnedSlot> g_pinned_free;
static bool pinned_acquire(PinnedSlot *out) {
    {
        std::lock_guard<std::mutex> lk(g_pinned_mu);
        if (!g_pinned_free.empty()) {
            *out = g_pinned_free.back();
            g_pinned_free.pop_back();
            return true;
        }
    }
    PinnedSlot s{nullptr, nullptr};
    if (cudaMallocHost((void **)&s.p, sizeof(DevHeader)) != cudaSuccess) { (void)cudaGetLastError(); return false; }
    if (cudaEventCreateWithFlags(&s.ev, cudaEventDisableTiming) != cudaSuccess) {
        (void)cudaGetLastError();
        cudaFreeHost(s.p);
        return false;
    }
    *out = s;
    return true;
}
static void pinned_release(DevHeader *p, cudaEvent_t ev) {
    if (!p) return;
    std::lock_guard<std::mutex> lk(g_pinned_mu);
    g_pinned_free.push_back(PinnedSlot{p, ev});
}

extern "C" int hdt_build_index(const int8_t *level, const int32_t *parent, const int32_t *cu_seqlens,
                               int32_t batch, int32_t total_tokens, const hdt_index_params_t *params,
                               void *workspace, size_t workspace_bytes, void *stream, hdt_index_t **out) {
    if (out) *out = nullptr;
    int bm, ms, bmu;
    norm_params(params, bm, ms, bmu);
    const int dirs = norm_dirs(params);
    if (!out || !cu_seqlens || !workspace || batch < 0 || total_tokens < 0 ||
        (total_tokens > 0 && (!level || !parent)))
        return set_error(HDT_ERR_INVALID_ARG, "hdt_build_index: null pointer or negative size");
    if (bm < 1 || bm > 128 || bmu < 1 || bmu > 128 || ms < 1 || ms > HDT_MAX_STAGES)
        return set_error(HDT_ERR_INVALID_ARG, "hdt_build_index: block_m, block_m_upper must be 1..128, max_stages 1..%d",
                         HDT_MAX_STAGES);
    if (params && (params->mask_off & ~7))
        return set_error(HDT_ERR_INVALID_ARG, "hdt_build_index: mask_off has bits outside 0..7");
    if (((uintptr_t)workspace & 255) != 0)
        return set_error(HDT_ERR_INVALID_ARG, "hdt_build_index: workspace must be 256-byte aligned");
    const int B = batch, T = total_tokens;
    const Layout L = make_layout(B, T, min(bm, bmu), ms);
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
    ix->batch = B; ix->total_tokens = T; ix->block_m = bm; ix->block_m_upper = bmu; ix->n_stages = 0;
    ix->directions = dirs;
    ix->workspace = workspace; ix->workspace_bytes = workspace_bytes;
    ix->rank = (const int *)(ws + L.rank);
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

    const int nel = max(T, B + 1);
    const int g_el = (nel + 255) / 256;
    const int g_chunk = max(1, (T + CHUNK - 1) / CHUNK);
    const int g_stride = max(1, min((T + 255) / 256, 148 * 8));
    static const int kSmemCap = 200 * 1024;
    static DevOnce attr_done;
    if (!attr_done.done()) {
        HDT_BUILD_CHECK(cudaFuncSetAttribute(k_walk, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemCap));
        HDT_BUILD_CHECK(cudaFuncSetAttribute(k_upper_stages, cudaFuncAttributeMaxDynamicSharedMemorySize, USMEM));
        attr_done.set();
    }
    // One CTA builds all stages above 0 when they are small (documents: a few percent of the
    // tokens, up to 3-4 stages).  A caller that allows many stages expects deep trees, whose upper
    // stages hold most of the elements: those go through the per-stage kernels.
    const bool fused_upper = (B <= UMAXB) && ms <= 8;
    // The upper stages only need stage 0's compaction; with their own scratch they are built on the
    // side stream while stage 0's blocks and queues are built on the caller's stream.
    Side *sd = nullptr;
    if (ms > 1 && !g_no_overlap && get_side(&sd) != HDT_OK) sd = nullptr;
    // The per-stage kernels (deep trees, many sequences) as two chains: what the next stage waits for (counts,
    // ranges, scan, compaction) on the caller's stream, the stage's blocks and queues (walk, block records,
    // ranking), which nothing but the attention kernels reads, on the side stream behind the stage's compaction.
    // The two share the family positions and the block scratch, so those alternate between two sets by stage
    // parity, and stage s + 2 takes a set only when the walk of stage s has read it.
    const bool piped = !fused_upper && sd != nullptr && ms > 1;

    // Everything the build enqueues; returns the first CUDA error.  Called directly or under
    // stream capture (see below).
    int n_launched = 0;
    auto enqueue_all = [&]() -> cudaError_t {
        cudaError_t e;
#define HDT_ENQ(expr) do { e = (expr); if (e != cudaSuccess) return e; } while (0)
        // header, cnt and nlc are adjacent in the workspace: one memset clears all three
        HDT_ENQ(cudaMemsetAsync(ws + L.header, 0, L.pre - L.header, st));
        k_init<<<g_el, 256, 0, st>>>(level, parent, cu_seqlens, B, T, HDT_MAX_STAGES * 8, hdr, ix->st[0].tok,
                                     ix->st[0].par, ix->st[0].scu, cnt, nlc);
        ++n_launched;
        auto launch_upper = [&](cudaStream_t s_) {
            UpperArgs u;
            for (int i = 0; i < HDT_MAX_STAGES; ++i) u.st[i] = ix->st[i < ms ? i : ms - 1];
            u.max_stages = ms; u.B = B; u.bm = bmu; u.dirs = dirs;
            u.cnt = cnt; u.nlc = nlc; u.pre = pre; u.keep = keep;
            u.bstart = (int *)(ws + L.bstart2); u.seqcount = (int *)(ws + L.seqcount2);
            u.fpos = (uint8_t *)(ws + L.fpos2); u.cost = (long long *)(ws + L.cost2);
            u.rank = (int *)(ws + L.rank);
            k_upper_stages<<<1, UT, USMEM, s_>>>(hdr, u);
            ++n_launched;
        };
        for (int s = 0; s < ms; ++s) {
            if (s >= 1 && fused_upper) {
                if (sd) HDT_ENQ(cudaStreamWaitEvent(st, sd->join, 0));
                else launch_upper(st);
                break;
            }
            // (piped: the scratch set of this stage's parity)
            const bool set2 = piped && (s & 1);
            uint8_t *fpos_s = set2 ? (uint8_t *)(ws + L.fpos2) : fpos;
            int *bstart_s = set2 ? (int *)(ws + L.bstart2) : bstart, *seqcount_s = set2 ? (int *)(ws + L.seqcount2) : seqcount;
            long long *cost_s = set2 ? (long long *)(ws + L.cost2) : cost;
            if (piped && s >= 2) HDT_ENQ(cudaStreamWaitEvent(st, sd->stage_ev[2 * (s - 2) + 1], 0));   // the walk of stage s - 2 has read fpos
            const StagePtrs &P = ix->st[s];
            // the last possible stage writes its (unused) next-stage arrays into its own up/pre scratch
            const StagePtrs &N = ix->st[(s + 1 < ms) ? s + 1 : s];
            const bool last = (s + 1 == ms);
            // (a kernel chain per stage: the stage before counted this stage's children in its compaction)
            HDT_ENQ(launch_chain(k_ranges, dim3(g_chunk), dim3(CHUNK), 0, st, hdr, s, s == 0 ? level : (const int8_t *)nullptr, P.par, cnt, nlc,
                                 P.rng, keep, fpos_s, blocksum, dirs, s == 0 ? (const int *)nullptr : (const int *)P.tok, (int *)(ws + L.rank)));
            // tok2 of the last possible stage is never read: point it at scratch (pre is rewritten first)
            const bool chain = !fused_upper;     // (else the one-CTA builder counts for itself and expects cleared arrays)
            HDT_ENQ(launch_chain(k_scan, dim3(g_chunk), dim3(CHUNK), 0, st, hdr, s, L.nchunk, keep, blocksum, P.tok, pre, P.up,
                                 last ? cnt : N.tok, chain ? cnt : (int *)nullptr, chain ? nlc : (int *)nullptr));
            n_launched += 2;
            if (!last) {
                HDT_ENQ(launch_chain(k_compact, dim3(g_stride), dim3(256), 0, st, hdr, s, B, P.par, P.up, pre, P.scu, N.par, N.scu, cnt, nlc,
                                     chain ? 1 : 0));
                ++n_launched;
                if (s == 0 && sd && fused_upper) {   // fork: the upper stages start now
                    HDT_ENQ(cudaEventRecord(sd->fork, st));
                    HDT_ENQ(cudaStreamWaitEvent(sd->s, sd->fork, 0));
                    launch_upper(sd->s);
                    HDT_ENQ(cudaEventRecord(sd->join, sd->s));
                }
            }
            cudaStream_t sb = st;        // the stream of the stage's blocks and queues
            if (piped) {
                sb = sd->s;
                HDT_ENQ(cudaEventRecord(sd->stage_ev[2 * s], st));
                HDT_ENQ(cudaStreamWaitEvent(sb, sd->stage_ev[2 * s], 0));
            }
            if (B > 0) {
                int maxlen_smem = kSmemCap;  // sequences longer than this walk through global memory
                const int bms = (s == 0) ? bm : bmu;
                HDT_ENQ(launch_chain(k_walk, dim3(B), dim3(256), (size_t)kSmemCap, sb, hdr, s, bms, P.scu, fpos_s, bstart_s, seqcount_s, maxlen_smem));
                if (piped) HDT_ENQ(cudaEventRecord(sd->stage_ev[2 * s + 1], sb));
                const int gy = max(1, min(64, 2048 / max(B, 1)));   // enough CTAs to spread a few long sequences
                HDT_ENQ(launch_chain(k_blocks, dim3(B, gy), dim3(256), 0, sb, hdr, s, bms, B, P.scu, bstart_s, seqcount_s, P.rng, P.up, P.blocks, cost_s));
                HDT_ENQ(launch_chain(k_queue, dim3(max(1, min(L.capnb / 8 + 1, 148 * 4))), dim3(256), 0, sb, hdr, s, cost_s, P.blocks, P.queue, P.queue_split));
                n_launched += 3;
            } else if (piped) {
                HDT_ENQ(cudaEventRecord(sd->stage_ev[2 * s + 1], sb));
            }
        }
        if (piped) {      // the side chain joins the caller's stream
            HDT_ENQ(cudaEventRecord(sd->join, sd->s));
            HDT_ENQ(cudaStreamWaitEvent(st, sd->join, 0));
        }
        return cudaGetLastError();
#undef HDT_ENQ
    };

    {
        ProfScope ps(PROF_INDEX, st);
        // The build is a dozen tiny kernels: launching them one by one is slower than running them.
        // They are captured once into a CUDA graph, which is replayed while the same buffers, sizes
        // and parameters come back (a few cached graphs per host thread).
        struct GraphKey { const void *a, *b, *c, *w; int B, T, bm, ms, bmu, ov, dirs, pad; };   // no padding bytes: compared with memcmp
        struct GraphCache { GraphKey key; cudaGraphExec_t exec; int launches; bool valid; unsigned long long used; };
        // (a few entries, least recently used replaced: a loop that alternates between buffer sets replays instead of capturing again)
        constexpr int kGraphs = 4;
        static thread_local GraphCache cache[kGraphs]{};
        static thread_local unsigned long long tick = 0;
        const GraphKey key{level, parent, cu_seqlens, workspace, B, T, bm, ms, bmu, sd ? 1 : 0, dirs, 0};
        static_assert(sizeof(GraphKey) == 4 * sizeof(void *) + 8 * sizeof(int), "GraphKey must not contain padding");
        bool done = false;
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        // (the legacy and per-thread default streams cannot be captured)
        const bool capturable = st != nullptr && st != cudaStreamLegacy && st != cudaStreamPerThread;
        if (!g_no_graph && capturable && cudaStreamIsCapturing(st, &cap) == cudaSuccess &&
            cap == cudaStreamCaptureStatusNone) {
            GraphCache *hit = nullptr, *victim = &cache[0];
            for (int i = 0; i < kGraphs; ++i) {
                if (cache[i].valid && std::memcmp(&cache[i].key, &key, sizeof(key)) == 0) hit = &cache[i];
                if (!cache[i].valid || (victim->valid && cache[i].used < victim->used)) victim = &cache[i];
            }
            if (hit) {
                hit->used = ++tick;
                if (cudaGraphLaunch(hit->exec, st) == cudaSuccess) { done = true; count_launch(hit->launches); }
            } else if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
                const cudaError_t e = enqueue_all();
                cudaGraph_t g = nullptr;
                const cudaError_t e2 = cudaStreamEndCapture(st, &g);
                cudaGraphExec_t exec = nullptr;
                if (e == cudaSuccess && e2 == cudaSuccess && g && cudaGraphInstantiate(&exec, g, 0) == cudaSuccess) {
                    if (victim->valid) cudaGraphExecDestroy(victim->exec);
                    *victim = GraphCache{key, exec, n_launched, true, ++tick};
                    if (cudaGraphLaunch(exec, st) == cudaSuccess) { done = true; count_launch(n_launched); }
                }
                if (g) cudaGraphDestroy(g);
                if (!done) (void)cudaGetLastError();   // fall back to direct launches below
            }
        }
        if (!done) {
            n_launched = 0;
            HDT_BUILD_CHECK(enqueue_all());
            count_launch(n_launched);
        }
    }
    // The header comes back through a pinned host buffer (a copy to pageable memory would be staged
    // by the driver).  First and last word of the buffer are set to a value the device never writes
    // (status is 0 or negative, tail is 0) so that the host can watch the copy land: it is the last
    // operation of the build on the stream, and its words arrive in order.
    PinnedSlot slot_{nullptr, nullptr};
    DevHeader *h_pinned = pinned_acquire(&slot_) ? slot_.p : nullptr;
    if (!h_pinned) {
        delete ix;
        return set_error(HDT_ERR_CUDA, "hdt_build_index: no pinned host memory for the index header");
    }
    // every word of the (reused) landing buffer is poisoned, not only the two the host watches
    for (size_t w = 0; w < sizeof(DevHeader) / sizeof(int); ++w) reinterpret_cast<int *>(h_pinned)[w] = kUnset;
    ix->h_pinned = h_pinned;
    ix->hdr_ev = slot_.ev;
    ix->hdr_dev = hdr;
    ix->stream = st;
    ix->max_stages = ms;
    ix->pending = 1;
    {
        // A deferred build leaves the caller's stream free for the attention kernel that follows: the
        // copy goes to the side stream, behind an event (the fallback wait of index_ready is then on
        // that stream).  Compute -> copy -> compute on one stream costs the kernel behind the copy a
        // few microseconds.
        cudaStream_t cs = st;
        Side *sdc = nullptr;
        if (params && params->deferred && !g_no_overlap && get_side(&sdc) == HDT_OK && sdc != nullptr &&
            cudaEventRecord(sdc->fork, st) == cudaSuccess && cudaStreamWaitEvent(sdc->s, sdc->fork, 0) == cudaSuccess) {
            cs = sdc->s;
            ix->stream = cs;
        }
        cudaError_t e_ = cudaMemcpyAsync(h_pinned, hdr, sizeof(DevHeader), cudaMemcpyDeviceToHost, cs);
        if (e_ == cudaSuccess) e_ = cudaEventRecord(slot_.ev, cs);      // the end of the copy, as the runtime sees it
        if (e_ != cudaSuccess) {
            (void)cudaStreamSynchronize(cs);                              // the copy may be queued: let it land first
            pinned_release(h_pinned, slot_.ev);
            delete ix;
            return set_error(HDT_ERR_CUDA, "queueing the copy of the index header failed: %s", cudaGetErrorString(e_));
        }
    }
#undef HDT_BUILD_CHECK
    if (!(params && params->deferred)) {
        const int rc = index_ready(ix);
        if (rc) {
            delete ix;
            return rc;
        }
    }
    *out = ix;
    return HDT_OK;
}

namespace hdt {
int index_ready(const hdt_index *cix) {
    hdt_index *ix = const_cast<hdt_index *>(cix);
    if (ix->pending) {
        // The host watches the copy land instead of sleeping in the driver: the first and the last
        // word of the buffer change when (parts of) the copy have arrived.  That is only a hint — the
        // bytes of one copy need not reach host memory in address order — so the event recorded
        // behind the copy decides: it is polled (about a microsecond per query) and, after a bounded
        // number of polls, waited for.
        DevHeader *hp = ix->h_pinned;
        volatile int *p_status = &hp->status, *p_tail = &hp->tail;
        bool landed = false;
        for (long long spin = 0; spin < 20000000LL && !landed; ++spin) landed = (*p_tail != kUnset && *p_status != kUnset);
        cudaError_t e_ = cudaErrorNotReady;
        for (int poll = 0; poll < 200000 && e_ == cudaErrorNotReady; ++poll) e_ = cudaEventQuery(ix->hdr_ev);
        if (e_ == cudaErrorNotReady) e_ = cudaEventSynchronize(ix->hdr_ev);
        if (e_ != cudaSuccess) {
            (void)cudaGetLastError();
            (void)cudaStreamSynchronize(ix->stream);
            ix->pending = 0;
            ix->failed = HDT_ERR_CUDA;
            pinned_release(hp, ix->hdr_ev);
            ix->h_pinned = nullptr;
            return set_error(HDT_ERR_CUDA, "waiting for the index build failed: %s", cudaGetErrorString(e_));
        }
        std::atomic_thread_fence(std::memory_order_acquire);
        const DevHeader h = *hp;
        pinned_release(hp, ix->hdr_ev);
        ix->h_pinned = nullptr;
        ix->pending = 0;
        ix->failed = h.status;
        ix->err_pos = h.err_pos;
        if (h.status == 0) {
            int ns = 1;
            while (ns < ix->max_stages && h.st[ns].n > 0) ++ns;
            // (a last stage that found "has_next" without one being built cannot happen below max_stages)
            if (h.st[ns - 1].has_next && ns == ix->max_stages) {
                ix->failed = HDT_ERR_BAD_HIERARCHY;
                ix->err_pos = -1;
            } else {
                ix->n_stages = ns;
                ix->nnz = h.nnz;
                ix->visited = h.visited;
                for (int s = 0; s <= HDT_MAX_STAGES; ++s) ix->desc[s] = h.st[s];
            }
        }
    }
    if (ix->failed == 0) return HDT_OK;
    if (ix->failed == HDT_ERR_BAD_HIERARCHY && ix->err_pos < 0)
        return set_error(HDT_ERR_BAD_HIERARCHY, "hdt_build_index: hierarchy needs more than max_stages = %d stages",
                         ix->max_stages);
    return set_error(ix->failed, "hdt_build_index: structure arrays violate a precondition near element %d", ix->err_pos);
}
}  // namespace hdt

extern "C" int hdt_index_info(const hdt_index_t *ix, int32_t *n_stages, int64_t *nnz, int64_t *visited) {
    if (!ix) return set_error(HDT_ERR_INVALID_ARG, "hdt_index_info: null index");
    if (const int rc = index_ready(ix)) return rc;
    if (n_stages) *n_stages = ix->n_stages;
    if (nnz) *nnz = ix->nnz;
    if (visited) *visited = ix->visited;
    return HDT_OK;
}

extern "C" int hdt_index_export(const hdt_index_t *ix, int32_t stage, hdt_stage_view_t *v) {
    if (!ix || !v) return set_error(HDT_ERR_INVALID_ARG, "hdt_index_export: null argument");
    if (const int rc = index_ready(ix)) return rc;
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
    if (ix && ix->pending) (void)index_ready(ix);     // the header copy must not land in a recycled buffer
    delete ix;
    return HDT_OK;
}
