// C-ABI entry points of the attention passes, error text, launch counter.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <memory>
#include <mutex>
#include <vector>

#include "hdt_internal.cuh"

namespace hdt {

static thread_local char g_err[512] = "";
std::atomic<long long> g_launches{0};

int set_error(int code, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

// ---- optional event timing -------------------------------------------------------------------
struct ProfRec { int id; cudaEvent_t a, b; };
static std::mutex g_prof_mu;
static bool g_prof_on = false;
static std::vector<ProfRec> g_prof_recs;      // recorded since the last read
static std::vector<ProfRec> g_prof_pool;      // created, free
static double g_prof_ms[PROF_COUNT];
static long long g_prof_n[PROF_COUNT];

ProfScope::ProfScope(int id, cudaStream_t s, bool enabled) : slot(-1), st(s) {
    if (!g_prof_on || !enabled) return;
    std::lock_guard<std::mutex> lk(g_prof_mu);
    ProfRec r;
    if (!g_prof_pool.empty()) { r = g_prof_pool.back(); g_prof_pool.pop_back(); }
    else if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) return;
    r.id = id;
    cudaEventRecord(r.a, st);
    g_prof_recs.push_back(r);
    slot = (int)g_prof_recs.size() - 1;
}
ProfScope::~ProfScope() {
    if (slot < 0) return;
    std::lock_guard<std::mutex> lk(g_prof_mu);
    cudaEventRecord(g_prof_recs[slot].b, st);
}

// ---- device-side failure word -------------------------------------------------------------------
__device__ int g_device_status[4] = {0, 0, 0, 0};  // [0] first failure recorded by a kernel (hdt_status_t), 0 = none; [1] where (kernel << 8 | wait site), [2] its loop count

int *device_status_ptr() {
    int *p = nullptr;
    if (cudaGetSymbolAddress((void **)&p, g_device_status) != cudaSuccess) {
        set_error(HDT_ERR_CUDA, "cudaGetSymbolAddress(g_device_status) failed");
        return nullptr;
    }
    return p;
}

// ---- side stream: the stages above 0 run beside stage 0 -------------------------------------------
// Two non-blocking streams (odd and even stages: their kernels are independent and should all
// be resident before stage 0 fills the SMs) and three events per host thread and device, created
// on first use.
static thread_local Side g_side[64];
int g_no_overlap = 0;
int g_no_graph = 0;
int g_phase_stamps = 0;
int g_no_fwd_mc = 0;
int g_no_pdl = 0;
static int g_no_multi_upper = 0;
static int g_no_self_beside = 0;
static int g_no_fused_delta = 0;
static int g_no_fold = 0;

int get_side(Side **out) {
    int dev = -1;
    HDT_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return set_error(HDT_ERR_UNSUPPORTED, "device ordinal %d", dev);
    Side &sd = g_side[dev];
    if (!sd.ready) {
        HDT_CUDA_CHECK(cudaStreamCreateWithFlags(&sd.s, cudaStreamNonBlocking));
        HDT_CUDA_CHECK(cudaStreamCreateWithFlags(&sd.s2, cudaStreamNonBlocking));
        HDT_CUDA_CHECK(cudaStreamCreateWithFlags(&sd.s3, cudaStreamNonBlocking));
        HDT_CUDA_CHECK(cudaEventCreateWithFlags(&sd.join3, cudaEventDisableTiming));
        HDT_CUDA_CHECK(cudaEventCreateWithFlags(&sd.fork, cudaEventDisableTiming));
        HDT_CUDA_CHECK(cudaEventCreateWithFlags(&sd.join, cudaEventDisableTiming));
        HDT_CUDA_CHECK(cudaEventCreateWithFlags(&sd.join2, cudaEventDisableTiming));
        HDT_CUDA_CHECK(cudaEventCreateWithFlags(&sd.fork0, cudaEventDisableTiming));
        HDT_CUDA_CHECK(cudaEventCreateWithFlags(&sd.join0, cudaEventDisableTiming));
        for (int i = 0; i < 2 * HDT_MAX_STAGES; ++i) HDT_CUDA_CHECK(cudaEventCreateWithFlags(&sd.stage_ev[i], cudaEventDisableTiming));
        sd.ready = true;
    }
    *out = &sd;
    return HDT_OK;
}

int sm_count(int *n_sm) {
    static std::atomic<int> cache[64];
    int dev = 0;
    HDT_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return set_error(HDT_ERR_UNSUPPORTED, "device ordinal %d", dev);
    int n = cache[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        HDT_CUDA_CHECK(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
        cache[dev].store(n, std::memory_order_relaxed);
    }
    *n_sm = n;
    return HDT_OK;
}

static size_t al256(size_t x) { return (x + 255) & ~size_t(255); }

struct AttnLayout {
    size_t delta;                       // bwd only
    size_t dq_acc;                      // bwd, bf16, head_dim 64, batches with split families: fp32 [T, H, 64] sums of dQ tiles
    bool has_dq_acc;
    size_t part[HDT_MAX_STAGES][4];     // partials handed from stage s-1 to stage s.  fwd: o, lse;  bwd: dq, dk, dv
    size_t own[HDT_MAX_STAGES][4];      // own partials of stage s when it is computed beside stage 0
    size_t total;
};

int g_bwd_walk = 0;                     // option "bwd_walk"

// Blocks of stage 0 that are neither self-contained nor EMPTY: families longer than a row block.
static int n_split_blocks(const hdt_index *ix) { return ix->desc[0].nb - ix->desc[0].n_fused - ix->desc[0].n_empty; }

static AttnLayout attn_layout(const hdt_index *ix, int H, int D, int bwd, int dtype = HDT_BF16) {
    AttnLayout L{};
    size_t o = 0;
    if (bwd) { L.delta = o; o += al256(sizeof(float) * (size_t)H * ix->total_tokens); }
    if (bwd && dtype == HDT_BF16 && D == 64 && n_split_blocks(ix) > 0) {
        L.has_dq_acc = true;
        L.dq_acc = o;
        o += al256(sizeof(float) * (size_t)ix->total_tokens * H * 64);
    }
    for (int s = 1; s < ix->n_stages; ++s) {
        const size_t n = (size_t)ix->desc[s].n;
        const int cnt = bwd ? 3 : 1;
        for (int c = 0; c < cnt; ++c) { L.part[s][c] = o; o += al256(sizeof(float) * n * H * D); }
        if (!bwd) { L.part[s][1] = o; o += al256(sizeof(float) * n * H); }
        for (int c = 0; c < cnt; ++c) { L.own[s][c] = o; o += al256(sizeof(float) * n * H * D); }
        if (!bwd) { L.own[s][1] = o; o += al256(sizeof(float) * n * H); }
    }
    L.total = o;
    return L;
}

static int check_common(const hdt_index *ix, int H, int D, int dtype, const void *ws, size_t ws_bytes,
                        size_t need, const char *fn) {
    if (!ix) return set_error(HDT_ERR_INVALID_ARG, "%s: null index", fn);
    if (H <= 0) return set_error(HDT_ERR_INVALID_ARG, "%s: heads must be positive", fn);
    if (D != 64 && D != 128) return set_error(HDT_ERR_UNSUPPORTED, "%s: head_dim %d not supported (64 or 128)", fn, D);
    if (dtype != HDT_F32 && dtype != HDT_BF16) return set_error(HDT_ERR_UNSUPPORTED, "%s: unknown dtype %d", fn, dtype);
    if (need > 0 && (!ws || ws_bytes < need))
        return set_error(HDT_ERR_WORKSPACE, "%s: workspace %zu < required %zu", fn, ws_bytes, need);
    if (need > 0 && ((uintptr_t)ws & 255) != 0)
        return set_error(HDT_ERR_INVALID_ARG, "%s: workspace must be 256-byte aligned", fn);
    return HDT_OK;
}

static bool misaligned(const void *p) { return ((uintptr_t)p & 15) != 0; }

}  // namespace hdt

using namespace hdt;

namespace hdt { int g_force_simt = 0; }
static int g_no_persistent = 0;
static int g_simt_upper = 0;

extern "C" int hdt_set_option(const char *name, int32_t value) {
    if (name && std::strcmp(name, "force_simt") == 0) { g_force_simt = value; return HDT_OK; }
    if (name && std::strcmp(name, "no_persistent") == 0) { g_no_persistent = value; return HDT_OK; }
    if (name && std::strcmp(name, "simt_upper") == 0) { g_simt_upper = value; return HDT_OK; }
    if (name && std::strcmp(name, "no_overlap") == 0) { g_no_overlap = value; return HDT_OK; }
    if (name && std::strcmp(name, "no_graph") == 0) { g_no_graph = value; return HDT_OK; }
    if (name && std::strcmp(name, "phase_stamps") == 0) { g_phase_stamps = value; return HDT_OK; }
    if (name && std::strcmp(name, "no_fused_delta") == 0) { g_no_fused_delta = value; return HDT_OK; }
    if (name && std::strcmp(name, "no_fold") == 0) { g_no_fold = value; return HDT_OK; }
    if (name && std::strcmp(name, "no_pdl") == 0) { g_no_pdl = value; return HDT_OK; }
    if (name && std::strcmp(name, "no_fwd_mc") == 0) { g_no_fwd_mc = value; return HDT_OK; }
    if (name && std::strcmp(name, "bwd_walk") == 0) { g_bwd_walk = value; return HDT_OK; }
    if (name && std::strcmp(name, "no_multi_upper") == 0) { g_no_multi_upper = value; return HDT_OK; }
    if (name && std::strcmp(name, "no_self_beside") == 0) { g_no_self_beside = value; return HDT_OK; }
    return set_error(HDT_ERR_INVALID_ARG, "hdt_set_option: unknown option");
}

extern "C" const char *hdt_last_error(void) { return g_err; }
extern "C" int64_t hdt_launch_count(void) { return (int64_t)g_launches.load(); }

// Waits for `stream`, then returns and clears the first failure recorded by a kernel.
extern "C" int hdt_device_status(void *stream) {
    HDT_CUDA_CHECK(cudaStreamSynchronize((cudaStream_t)stream));
    int h[4] = {0, 0, 0, 0};
    HDT_CUDA_CHECK(cudaMemcpyFromSymbol(h, g_device_status, sizeof(h)));
    if (h[0] != 0) {
        const int zero[4] = {0, 0, 0, 0};
        HDT_CUDA_CHECK(cudaMemcpyToSymbol(g_device_status, zero, sizeof(zero)));
        return set_error(h[0], "a kernel recorded device-side failure %d (a bounded wait ran out; kernel %d, wait %d, loop count %d)",
                         h[0], h[1] >> 8, h[1] & 255, h[2]);
    }
    return HDT_OK;
}

extern "C" int hdt_profile_enable(int32_t on) {
    std::lock_guard<std::mutex> lk(g_prof_mu);
    g_prof_on = on != 0;
    return HDT_OK;
}

extern "C" const char *hdt_profile_name(int32_t id) {
    static const char *names[PROF_COUNT] = {"index_build(all kernels)", "k_fwd_stage0", "k_fwd_upper_stages",
                                            "k_delta", "k_bwd_stage0", "k_bwd_upper_stages"};
    return (id >= 0 && id < PROF_COUNT) ? names[id] : "";
}

extern "C" int hdt_profile_read(int32_t id, int64_t *launches, double *total_ms, int32_t reset) {
    if (id < 0 || id >= PROF_COUNT) return set_error(HDT_ERR_INVALID_ARG, "hdt_profile_read: bad id %d", id);
    std::lock_guard<std::mutex> lk(g_prof_mu);
    for (ProfRec &r : g_prof_recs) {   // fold finished records into the totals
        HDT_CUDA_CHECK(cudaEventSynchronize(r.b));
        float ms = 0.f;
        HDT_CUDA_CHECK(cudaEventElapsedTime(&ms, r.a, r.b));
        g_prof_ms[r.id] += ms;
        g_prof_n[r.id] += 1;
        g_prof_pool.push_back(r);
    }
    g_prof_recs.clear();
    if (launches) *launches = g_prof_n[id];
    if (total_ms) *total_ms = g_prof_ms[id];
    if (reset) { g_prof_n[id] = 0; g_prof_ms[id] = 0.0; }
    return HDT_OK;
}

extern "C" size_t hdt_attn_workspace_bytes(const hdt_index_t *ix, int32_t heads, int32_t head_dim,
                                           int32_t dtype, int32_t bwd) {
    (void)dtype;
    if (!ix || heads <= 0 || head_dim <= 0) return 0;
    if (index_ready(ix)) return 0;
    return attn_layout(ix, heads, head_dim, bwd, dtype).total;
}

extern "C" int hdt_attn_fwd(const hdt_index_t *ix, const void *q, const void *k, const void *v, void *o,
                            float *lse, int32_t heads, int32_t head_dim, int32_t dtype, float softmax_scale,
                            void *workspace, size_t workspace_bytes, void *stream) {
    if (!ix) return set_error(HDT_ERR_INVALID_ARG, "hdt_attn_fwd: null index");
    int rc = check_common(ix, heads, head_dim, dtype, workspace, workspace_bytes, 0, "hdt_attn_fwd");
    if (rc) return rc;
    if (ix->total_tokens > 0) {
        if (!q || !k || !v || !o || !lse) return set_error(HDT_ERR_INVALID_ARG, "hdt_attn_fwd: null tensor pointer");
        if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(o))
            return set_error(HDT_ERR_INVALID_ARG, "hdt_attn_fwd: tensors must be 16-byte aligned");
    }
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
    cudaStream_t st = (cudaStream_t)stream;
    char *ws = (char *)workspace;
    int *status = device_status_ptr();
    if (!status) return HDT_ERR_CUDA;
    // A deferred index whose build is still in flight: the looping stage-0 kernel of bf16 calls is
    // queued before the host waits for the counts (it reads them on the device), so the GPU goes
    // from the build straight into the attention.  The stream is forked first: what the host
    // launches on the side streams after its wait still runs beside that kernel, not behind it.
    bool early = false;
    std::unique_ptr<ProfScope> ps_early;      // stage 0's time when a kernel goes ahead: from its start to the end of the stage's other kernel
    if (ix->pending && ix->total_tokens > 0 && dtype == HDT_BF16 && !g_force_simt && g_no_persistent == 0 &&
        !g_no_overlap && (workspace == nullptr || ((uintptr_t)workspace & 255) == 0)) {
        Side *sd = nullptr;
        rc = get_side(&sd);
        if (rc) return rc;
        HDT_CUDA_CHECK(cudaEventRecord(sd->fork, st));
        const StagePtrs &P = ix->st[0];
        FwdStageArgs a{};
        a.n = ix->total_tokens; a.H = heads; a.T = ix->total_tokens;
        a.rng = P.rng; a.up = P.up; a.blocks = P.blocks; a.queue = P.queue; a.queue_split = P.queue_split;
        a.block_rows = ix->block_m;
        a.q = q; a.k = k; a.v = v;
        a.scale_log2 = scale * 1.4426950408889634f;
        a.part_o = (float *)ws;              // stage 1's partial results come first in the workspace
        a.ws_bytes = workspace ? workspace_bytes : 0;
        a.hdr = ix->hdr_dev;
        a.o = o; a.lse = lse;
        a.status = status;
        a.dirs = ix->directions;
        a.part = 1;
        ps_early.reset(new ProfScope(PROF_FWD_STAGE0, st));
        rc = launch_fwd_tc(a, head_dim, st);
        if (rc) return rc;
        early = true;
    }
    rc = index_ready(ix);
    if (rc) return rc;
    const AttnLayout L = attn_layout(ix, heads, head_dim, 0);
    rc = check_common(ix, heads, head_dim, dtype, workspace, workspace_bytes, L.total, "hdt_attn_fwd");
    if (rc) return rc;
    if (ix->total_tokens == 0) return HDT_OK;
    auto stage_args = [&](int s) {
        const StagePtrs &P = ix->st[s];
        FwdStageArgs a{};
        a.n = ix->desc[s].n; a.nb = ix->desc[s].nb; a.H = heads; a.T = ix->total_tokens;
        a.tok = s ? P.tok : nullptr;
        a.rng = P.rng; a.up = P.up; a.blocks = P.blocks; a.queue = P.queue;
        a.queue_split = P.queue_split; a.n_fused = ix->desc[s].n_fused;
        a.n_empty = ix->desc[s].n_empty;
        a.block_rows = s ? ix->block_m_upper : ix->block_m;
        a.q = q; a.k = k; a.v = v;
        a.scale_log2 = scale * 1.4426950408889634f;
        if (s > 0) {   // partial results the stages below left for this stage's elements
            a.carry_o = (const float *)(ws + L.part[s][0]);
            a.carry_lse = (const float *)(ws + L.part[s][1]);
        }
        if (s + 1 < ix->n_stages) {   // where this stage leaves its own for the next one
            a.part_o = (float *)(ws + L.part[s + 1][0]);
            a.part_lse = (float *)(ws + L.part[s + 1][1]);
        }
        a.o = o; a.lse = lse;
        a.status = status;
        a.no_persistent = g_no_persistent;
        a.dirs = ix->directions;
        a.tok_rows = a.tok;
        return a;
    };
    // The stages above 0 do not depend on stage 0 until their results are merged: compute them on
    // the side stream while stage 0 runs, then finish each with an element-wise merge.
    const bool overlap = (ix->n_stages > 1 && !g_no_overlap) || early;
    if (overlap) {
        Side *sd = nullptr;
        rc = get_side(&sd);
        if (rc) return rc;
        if (!early) HDT_CUDA_CHECK(cudaEventRecord(sd->fork, st));
        HDT_CUDA_CHECK(cudaStreamWaitEvent(sd->s, sd->fork, 0));
        const bool tc0 = dtype == HDT_BF16 && !g_force_simt;
        // Stage 0's blocks that are not self-contained (split families, EMPTY blocks) have a kernel of
        // their own.  Where the split families are the smaller part it runs on the second side stream beside the
        // looping kernel (measured: a batch of padded documents gains 7 %); where split families
        // dominate, one kernel after the other is faster (the skewed batch loses 3 % side by side).
        const bool rest_beside = early || (tc0 && 2 * (ix->desc[0].nb - ix->desc[0].n_fused - ix->desc[0].n_empty) <= ix->desc[0].nb);
        const bool two = ix->n_stages > 2;
        if (two) HDT_CUDA_CHECK(cudaStreamWaitEvent(sd->s2, sd->fork, 0));
        // Stages above 0 of bf16 calls run on the gathering tensor-core kernels, whatever the depth of the
        // hierarchy (option "simt_upper" = 1: on the fp32 SIMT kernels, which take trees of more than three
        // stages in one launch over the blocks of all those stages).
        const bool tc_upper = dtype == HDT_BF16 && !g_force_simt && !g_simt_upper;
        ChainArgs c{};
        c.n1 = ix->desc[1].n; c.H = heads; c.T = ix->total_tokens; c.n_stages = ix->n_stages; c.nt = 1;
        c.tok1 = ix->st[1].tok;
        // On the gathering kernels stage 1 runs after stage 0 and completes its elements itself
        // (its own result merged with stage 0's partial and stage 2's own); only stage 2 runs beside
        // stage 0, and there is no merge kernel.  That pays while the stage-1 kernel is shorter than
        // the merge it saves (about 10 us): no family of stage 1 longer than a block, and its CTAs
        // resident at once.  Otherwise (skewed documents with long sections: 47 us against 13; large
        // batches at head_dim 128: 59 against 23) stage 1 runs beside stage 0 like the others and the
        // merge kernel follows.
        int n_sm1 = 0;
        if (const int rc_ = sm_count(&n_sm1)) return rc_;
        const bool short1 = ix->n_stages > 1 && ix->desc[1].n_fused + ix->desc[1].n_empty == ix->desc[1].nb &&
                            (long long)ix->desc[1].nb * heads <= 2LL * n_sm1;
        const bool fold = tc_upper && !(g_no_fold & 1) && (short1 || (g_no_fold & 2)) && ix->n_stages > 1 && ix->n_stages <= 3;
        FwdStageArgs a1{};
        // (deep trees on the SIMT kernels: the stages above 0 are independent in own-partial mode and small, and a
        // launch per stage is mostly launch latency: one launch over the blocks of all of them.  The tensor-core
        // kernels keep a launch per stage, odd and even stages on two streams: one launch over all their blocks
        // takes every SM ahead of stage 0 and was slower, 1.253 against 1.234 ms on the expression trees.)
        const bool multi = !tc_upper && ix->n_stages > 3 && !g_no_multi_upper;
        MultiFwdArgs mf{};
        for (int s = 1; s < ix->n_stages; ++s) {
            FwdStageArgs a = stage_args(s);
            a.own_o = (float *)(ws + L.own[s][0]);
            a.own_lse = (float *)(ws + L.own[s][1]);
            c.up[s] = ix->st[s].up; c.own[s][0] = a.own_o; c.own_lse[s] = a.own_lse;
            if (fold && s == 1) { a1 = a; continue; }
            if (multi) {
                if (mf.n == 0) { mf.base = a; mf.base.carry_o = nullptr; mf.base.carry_lse = nullptr; mf.base.part_o = nullptr; mf.base.part_lse = nullptr; }
                MultiStage &t = mf.st[mf.n];
                t.n = a.n; t.nb = a.nb; t.cum = mf.n ? mf.st[mf.n - 1].cum + mf.st[mf.n - 1].nb : 0;
                t.tok = a.tok; t.rng = a.rng; t.up = a.up; t.blocks = a.blocks; t.queue = a.queue;
                t.own[0] = a.own_o; t.own_lse = a.own_lse;
                ++mf.n;
                continue;
            }
            cudaStream_t ss = (s & 1) ? sd->s : sd->s2;
            if (tc_upper) rc = launch_fwd_tc_upper(a, head_dim, ss);
            else rc = launch_fwd_simt(a, head_dim, dtype, ss);
            if (rc) return rc;
        }
        if (multi) {
            rc = launch_fwd_simt_multi(mf, head_dim, dtype, sd->s);
            if (rc) return rc;
        }
        if (rest_beside) {
            FwdStageArgs a = stage_args(0);
            a.part = 2;
            // On a stream of its own, queued after the stages above 0: their CTAs are dispatched first as SMs
            // become free, and this kernel does not wait for any of them to finish.
            HDT_CUDA_CHECK(cudaStreamWaitEvent(sd->s3, sd->fork, 0));
            rc = launch_fwd_tc(a, head_dim, sd->s3);
            if (rc) return rc;
        }
        HDT_CUDA_CHECK(cudaEventRecord(sd->join, sd->s));
        if (two) HDT_CUDA_CHECK(cudaEventRecord(sd->join2, sd->s2));
        if (rest_beside) HDT_CUDA_CHECK(cudaEventRecord(sd->join3, sd->s3));
        {   // stage 0 after the small side kernels are queued: they take their SM share first (the
            // stage-0 kernel would otherwise fill every SM and push them behind itself)
            FwdStageArgs a = stage_args(0);
            a.part = rest_beside ? 1 : 0;
            if (!early) {                    // (early: already queued)
                ProfScope ps(PROF_FWD_STAGE0, st);
                if (tc0) rc = launch_fwd_tc(a, head_dim, st);
                else rc = launch_fwd_simt(a, head_dim, dtype, st);
                if (rc) return rc;
            }
        }
        if (ix->n_stages == 1) {             // (early only) nothing to merge: wait for the other blocks' kernel
            if (two) HDT_CUDA_CHECK(cudaStreamWaitEvent(st, sd->join2, 0));
            if (rest_beside) HDT_CUDA_CHECK(cudaStreamWaitEvent(st, sd->join3, 0));
            ps_early.reset();
            return HDT_OK;
        }
        if (rest_beside) HDT_CUDA_CHECK(cudaStreamWaitEvent(st, sd->join3, 0));
        ps_early.reset();                    // (stage 0 ends here: both of its kernels are done)
        HDT_CUDA_CHECK(cudaStreamWaitEvent(st, sd->join, 0));
        if (two) HDT_CUDA_CHECK(cudaStreamWaitEvent(st, sd->join2, 0));
        ProfScope ps(PROF_FWD_UPPER, st);
        if (fold) {
            a1.final_merge = 1;
            a1.own_o = nullptr; a1.own_lse = nullptr;
            if (ix->n_stages > 2) { a1.next_own_o = c.own[2][0]; a1.next_own_lse = c.own_lse[2]; }
            return launch_fwd_tc_upper(a1, head_dim, st);
        }
        c.base[0] = (const float *)(ws + L.part[1][0]);
        c.base_lse = (const float *)(ws + L.part[1][1]);
        c.out[0] = o; c.lse = lse;
        return launch_chain_merge(c, head_dim, dtype, st);
    }
    for (int s = 0; s < ix->n_stages; ++s) {   // bottom-up: stage 0 first
        FwdStageArgs a = stage_args(s);
        {
            ProfScope ps(s == 0 ? PROF_FWD_STAGE0 : PROF_FWD_UPPER, st);
            if (s == 0 && dtype == HDT_BF16 && !g_force_simt) rc = launch_fwd_tc(a, head_dim, st);
            else rc = launch_fwd_simt(a, head_dim, dtype, st);
        }
        if (rc) return rc;
    }
    return HDT_OK;
}

extern "C" int hdt_attn_bwd(const hdt_index_t *ix, const void *q, const void *k, const void *v, const void *o,
                            const float *lse, const void *d_o, void *dq, void *dk, void *dv, int32_t heads,
                            int32_t head_dim, int32_t dtype, float softmax_scale, void *workspace,
                            size_t workspace_bytes, void *stream) {
    if (!ix) return set_error(HDT_ERR_INVALID_ARG, "hdt_attn_bwd: null index");
    if (const int rc0 = index_ready(ix)) return rc0;
    const AttnLayout L = attn_layout(ix, heads > 0 ? heads : 1, head_dim > 0 ? head_dim : 64, 1, dtype);
    int rc = check_common(ix, heads, head_dim, dtype, workspace, workspace_bytes, L.total, "hdt_attn_bwd");
    if (rc) return rc;
    if (ix->total_tokens == 0) return HDT_OK;
    if (!q || !k || !v || !o || !lse || !d_o || !dq || !dk || !dv)
        return set_error(HDT_ERR_INVALID_ARG, "hdt_attn_bwd: null tensor pointer");
    if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(o) || misaligned(d_o) || misaligned(dq) ||
        misaligned(dk) || misaligned(dv))
        return set_error(HDT_ERR_INVALID_ARG, "hdt_attn_bwd: tensors must be 16-byte aligned");
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
    cudaStream_t st = (cudaStream_t)stream;
    char *ws = (char *)workspace;
    float *delta = (float *)(ws + L.delta);
    int *status = device_status_ptr();
    if (!status) return HDT_ERR_CUDA;
    const bool overlap = ix->n_stages > 1 && !g_no_overlap;
    // Stages above 0 of bf16 calls: the gathering tensor-core kernels (see hdt_attn_fwd).
    const bool tc_upper = dtype == HDT_BF16 && !g_force_simt && !g_simt_upper;
    // No delta pass when every kernel of this call computes dO . O of its rows itself: stage 0
    // entirely on the looping kernels (the transposed one at head_dim 64, the fused five-MMA one at
    // head_dim 128; every block self-contained), the stages above it on the gathering tensor-core kernels.
    const bool fused_delta = dtype == HDT_BF16 && !g_force_simt && (head_dim == 64 || head_dim == 128) && g_no_persistent == 0 &&
                             !g_no_fused_delta && ix->directions == 7 && ix->desc[0].n_fused == ix->desc[0].nb &&
                             ix->desc[0].nb > 0 && (ix->n_stages == 1 || (overlap && tc_upper));
    // Families longer than a row block (head_dim 64): one walk over their tile pairs, dQ tiles summed
    // in an fp32 buffer that starts at zero (option "bwd_walk" = 1: two walks, no buffer).
    float *dq_acc = nullptr;
    if (L.has_dq_acc && !g_force_simt && g_bwd_walk != 1 &&
        (g_no_persistent == 0 || g_no_persistent == 4 || g_no_persistent == 6)) {
        dq_acc = (float *)(ws + L.dq_acc);
    }
    // The buffer is cleared (writes) beside the delta pass (reads), on the second side stream: both are
    // HBM-bound, one in each direction.  Stage 0 waits for it (join0).
    Side *sd0 = nullptr;
    const bool clear_beside = dq_acc != nullptr && !fused_delta && !g_no_overlap && get_side(&sd0) == HDT_OK && sd0 != nullptr;
    if (dq_acc != nullptr) {
        const size_t bytes = sizeof(float) * (size_t)ix->total_tokens * heads * 64;
        if (clear_beside) {
            HDT_CUDA_CHECK(cudaEventRecord(sd0->fork0, st));
            HDT_CUDA_CHECK(cudaStreamWaitEvent(sd0->s2, sd0->fork0, 0));
            HDT_CUDA_CHECK(cudaMemsetAsync(dq_acc, 0, bytes, sd0->s2));
            HDT_CUDA_CHECK(cudaEventRecord(sd0->join0, sd0->s2));
        } else {
            ProfScope ps(PROF_BWD_STAGE0, st);
            HDT_CUDA_CHECK(cudaMemsetAsync(dq_acc, 0, bytes, st));
        }
    }
    if (!fused_delta) {
        ProfScope ps(PROF_DELTA, st);
        rc = launch_delta(o, d_o, delta, ix->total_tokens, heads, head_dim, dtype, st);
    }
    if (rc) return rc;
    if (clear_beside) HDT_CUDA_CHECK(cudaStreamWaitEvent(st, sd0->join0, 0));
    auto stage_args = [&](int s) {
        const StagePtrs &P = ix->st[s];
        BwdStageArgs a{};
        a.n = ix->desc[s].n; a.nb = ix->desc[s].nb; a.H = heads; a.T = ix->total_tokens;
        a.tok = s ? P.tok : nullptr;
        a.rng = P.rng; a.up = P.up; a.blocks = P.blocks; a.queue = P.queue;
        a.queue_split = P.queue_split; a.n_fused = ix->desc[s].n_fused;
        a.block_rows = s ? ix->block_m_upper : ix->block_m;
        a.q = q; a.k = k; a.v = v; a.d_o = d_o; a.lse = lse; a.delta = fused_delta ? nullptr : delta; a.o = o;
        a.scale = scale;
        a.scale_log2 = scale * 1.4426950408889634f;
        if (s > 0) {
            a.carry_dq = (const float *)(ws + L.part[s][0]);
            a.carry_dk = (const float *)(ws + L.part[s][1]);
            a.carry_dv = (const float *)(ws + L.part[s][2]);
        }
        if (s + 1 < ix->n_stages) {
            a.part_dq = (float *)(ws + L.part[s + 1][0]);
            a.part_dk = (float *)(ws + L.part[s + 1][1]);
            a.part_dv = (float *)(ws + L.part[s + 1][2]);
        }
        a.dq = dq; a.dk = dk; a.dv = dv;
        a.status = status;
        a.no_persistent = g_no_persistent;
        a.dirs = ix->directions;
        a.tok_rows = a.tok;
        if (s == 0) a.dq_acc = dq_acc;
        a.n_empty = ix->desc[s].n_empty;
        return a;
    };
    if (overlap) {   // delta is ready: the upper stages' own gradients are computed beside stage 0
        Side *sd = nullptr;
        rc = get_side(&sd);
        if (rc) return rc;
        HDT_CUDA_CHECK(cudaEventRecord(sd->fork, st));
        HDT_CUDA_CHECK(cudaStreamWaitEvent(sd->s, sd->fork, 0));
        // (with the one-walk kernel the self-contained blocks' kernel goes to the second side stream: its CTAs take
        // the SMs that the one-walk kernel's CTAs leave first, and it shares HBM with the pass that converts dQ)
        const bool self_beside = dq_acc != nullptr && ix->desc[0].n_fused > 0 && !g_no_self_beside;
        const bool two = ix->n_stages > 2 || self_beside;
        if (two) HDT_CUDA_CHECK(cudaStreamWaitEvent(sd->s2, sd->fork, 0));
        ChainArgs c{};
        c.n1 = ix->desc[1].n; c.H = heads; c.T = ix->total_tokens; c.n_stages = ix->n_stages; c.nt = 3;
        c.tok1 = ix->st[1].tok;
        // (stage 1 on the gathering kernels: after stage 0, completing its elements itself; see hdt_attn_fwd)
        const bool fold = tc_upper && (g_no_fold & 4) && ix->n_stages <= 3;   // measured: no gain in the backward (the kernel is longer than the merge it saves); option only
        BwdStageArgs a1{};
        const bool multi = !tc_upper && ix->n_stages > 3 && !g_no_multi_upper;      // (see hdt_attn_fwd)
        MultiBwdArgs mb{};
        for (int s = 1; s < ix->n_stages; ++s) {
            BwdStageArgs a = stage_args(s);
            a.own_dq = (float *)(ws + L.own[s][0]);
            a.own_dk = (float *)(ws + L.own[s][1]);
            a.own_dv = (float *)(ws + L.own[s][2]);
            c.up[s] = ix->st[s].up;
            c.own[s][0] = a.own_dq; c.own[s][1] = a.own_dk; c.own[s][2] = a.own_dv;
            if (fold && s == 1) { a1 = a; continue; }
            if (multi) {
                if (mb.n == 0) {
                    mb.base = a;
                    mb.base.carry_dq = nullptr; mb.base.carry_dk = nullptr; mb.base.carry_dv = nullptr;
                    mb.base.part_dq = nullptr; mb.base.part_dk = nullptr; mb.base.part_dv = nullptr;
                }
                MultiStage &t = mb.st[mb.n];
                t.n = a.n; t.nb = a.nb; t.cum = mb.n ? mb.st[mb.n - 1].cum + mb.st[mb.n - 1].nb : 0;
                t.tok = a.tok; t.rng = a.rng; t.up = a.up; t.blocks = a.blocks; t.queue = a.queue;
                t.own[0] = a.own_dq; t.own[1] = a.own_dk; t.own[2] = a.own_dv;
                ++mb.n;
                continue;
            }
            cudaStream_t ss = (s & 1) ? sd->s : sd->s2;
            if (tc_upper) rc = launch_bwd_tc_upper(a, head_dim, ss);
            else rc = launch_bwd_simt(a, head_dim, dtype, ss);
            if (rc) return rc;
        }
        if (multi) {
            rc = launch_bwd_simt_multi(mb, head_dim, dtype, sd->s);
            if (rc) return rc;
        }
        HDT_CUDA_CHECK(cudaEventRecord(sd->join, sd->s));
        if (two && !self_beside) HDT_CUDA_CHECK(cudaEventRecord(sd->join2, sd->s2));
        {
            BwdStageArgs a = stage_args(0);
            if (self_beside) a.self_stream = (void *)sd->s2;
            ProfScope ps(PROF_BWD_STAGE0, st);
            if (dtype == HDT_BF16 && !g_force_simt) rc = launch_bwd_tc(a, head_dim, st);
            else rc = launch_bwd_simt(a, head_dim, dtype, st);
            if (rc) return rc;
            if (self_beside) {       // (inside the scope: stage 0 ends when both streams have)
                HDT_CUDA_CHECK(cudaEventRecord(sd->join2, sd->s2));
                HDT_CUDA_CHECK(cudaStreamWaitEvent(st, sd->join2, 0));
            }
        }
        HDT_CUDA_CHECK(cudaStreamWaitEvent(st, sd->join, 0));
        if (two && !self_beside) HDT_CUDA_CHECK(cudaStreamWaitEvent(st, sd->join2, 0));
        ProfScope ps(PROF_BWD_UPPER, st);
        if (fold) {
            a1.final_merge = 1;
            a1.own_dq = nullptr; a1.own_dk = nullptr; a1.own_dv = nullptr;
            if (ix->n_stages > 2) {
                a1.next_own_dq = c.own[2][0]; a1.next_own_dk = c.own[2][1]; a1.next_own_dv = c.own[2][2];
            }
            return launch_bwd_tc_upper(a1, head_dim, st);
        }
        for (int k = 0; k < 3; ++k) c.base[k] = (const float *)(ws + L.part[1][k]);
        c.out[0] = dq; c.out[1] = dk; c.out[2] = dv;
        return launch_chain_merge(c, head_dim, dtype, st);
    }
    for (int s = 0; s < ix->n_stages; ++s) {   // bottom-up: stage 0 first
        BwdStageArgs a = stage_args(s);
        {
            ProfScope ps(s == 0 ? PROF_BWD_STAGE0 : PROF_BWD_UPPER, st);
            if (s == 0 && dtype == HDT_BF16 && !g_force_simt) rc = launch_bwd_tc(a, head_dim, st);
            else rc = launch_bwd_simt(a, head_dim, dtype, st);
        }
        if (rc) return rc;
    }
    return HDT_OK;
}

// ---------------------------------------------------------------------------------------------
// Forward pass for callers that cannot allocate device memory
// ---------------------------------------------------------------------------------------------
// The partial results of the upper stages normally live in a workspace the caller allocates.
// Here they live in this fixed array, which every GPU that loads the library holds until the
// process exits.  In host code the name `g_fwd_scratch` is only a handle: the device address
// comes from cudaGetSymbolAddress, once per device, with that device current.
#define HDT_FWD_STATIC_SCRATCH_BYTES (8u << 20)
static __device__ __align__(256) unsigned char g_fwd_scratch[HDT_FWD_STATIC_SCRATCH_BYTES];

static void *g_fwd_scratch_ptr[64];   // device address of g_fwd_scratch, per device ordinal
static std::mutex g_fwd_scratch_mu;

extern "C" size_t hdt_attn_fwd_static_max_bytes(void) { return (size_t)HDT_FWD_STATIC_SCRATCH_BYTES; }

extern "C" int hdt_attn_fwd_static(const hdt_index_t *ix, const void *q, const void *k, const void *v, void *o,
                                   float *lse, int32_t heads, int32_t head_dim, int32_t dtype,
                                   float softmax_scale, void *stream) {
    if (!ix) return set_error(HDT_ERR_INVALID_ARG, "hdt_attn_fwd_static: null index");
    if (const int rc0 = index_ready(ix)) return rc0;
    const AttnLayout L = attn_layout(ix, heads > 0 ? heads : 1, head_dim > 0 ? head_dim : 64, 0);
    if (L.total > (size_t)HDT_FWD_STATIC_SCRATCH_BYTES)
        return set_error(HDT_ERR_WORKSPACE,
                         "hdt_attn_fwd_static: this batch needs %zu bytes of scratch, the built-in array holds %zu; "
                         "use hdt_attn_fwd with a caller workspace",
                         L.total, (size_t)HDT_FWD_STATIC_SCRATCH_BYTES);
    int dev = -1;
    HDT_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return set_error(HDT_ERR_UNSUPPORTED, "hdt_attn_fwd_static: device ordinal %d", dev);
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lk(g_fwd_scratch_mu);
        if (!g_fwd_scratch_ptr[dev]) {   // first call on this device: resolve the array's device address
            void *p = nullptr;
            HDT_CUDA_CHECK(cudaGetSymbolAddress(&p, g_fwd_scratch));
            g_fwd_scratch_ptr[dev] = p;
        }
        scratch = g_fwd_scratch_ptr[dev];
    }
    int rc = check_common(ix, heads, head_dim, dtype, scratch, (size_t)HDT_FWD_STATIC_SCRATCH_BYTES, L.total,
                          "hdt_attn_fwd_static");
    if (rc) return rc;
    if (ix->total_tokens == 0) return HDT_OK;
    if (!q || !k || !v || !o || !lse)
        return set_error(HDT_ERR_INVALID_ARG, "hdt_attn_fwd_static: null tensor pointer");
    if (misaligned(q) || misaligned(k) || misaligned(v) || misaligned(o))
        return set_error(HDT_ERR_INVALID_ARG, "hdt_attn_fwd_static: tensors must be 16-byte aligned");
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
    cudaStream_t st = (cudaStream_t)stream;
    char *ws = (char *)scratch;
    int *status = device_status_ptr();
    if (!status) return HDT_ERR_CUDA;
    // Every partial result a stage reads was written by the stage below it in this same call, so
    // nothing in the array has to start at zero; what the previous call left is overwritten.
    for (int s = 0; s < ix->n_stages; ++s) {   // bottom-up: stage 0 first
        const StagePtrs &P = ix->st[s];
        FwdStageArgs a{};
        a.n = ix->desc[s].n; a.nb = ix->desc[s].nb; a.H = heads; a.T = ix->total_tokens;
        a.tok = s ? P.tok : nullptr;
        a.rng = P.rng; a.up = P.up; a.blocks = P.blocks; a.queue = P.queue;
        a.queue_split = P.queue_split; a.n_fused = ix->desc[s].n_fused;
        a.block_rows = s ? ix->block_m_upper : ix->block_m;
        a.q = q; a.k = k; a.v = v;
        a.scale_log2 = scale * 1.4426950408889634f;
        if (s > 0) {   // partial results the stages below left for this stage's elements
            a.carry_o = (const float *)(ws + L.part[s][0]);
            a.carry_lse = (const float *)(ws + L.part[s][1]);
        }
        if (s + 1 < ix->n_stages) {   // where this stage leaves its own for the next one
            a.part_o = (float *)(ws + L.part[s + 1][0]);
            a.part_lse = (float *)(ws + L.part[s + 1][1]);
        }
        a.o = o; a.lse = lse;
        a.status = status;
        a.no_persistent = g_no_persistent;
        a.dirs = ix->directions;
        a.tok_rows = a.tok;
        if (s == 0 && dtype == HDT_BF16 && !g_force_simt) rc = launch_fwd_tc(a, head_dim, st);
        else rc = launch_fwd_simt(a, head_dim, dtype, st);
        if (rc) return rc;
    }
    return HDT_OK;
}
