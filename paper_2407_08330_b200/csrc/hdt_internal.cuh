// Internal declarations shared by the translation units of libhdt.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <atomic>

#include "../../include/hdt.h"
#include "../../include/hdt_debug.h"

namespace hdt {

// Device-resident header of an index (first bytes of the index workspace).
struct StageDesc {
    int n;         // elements of the stage array
    int nb;        // row blocks
    int has_next;  // a later stage exists
    int n_fused;   // blocks that are SELF and not EMPTY (first n_fused entries of queue_split)
    int n_empty;   // EMPTY blocks (rows without any key in this stage: PAD, lone roots)
};

struct DevHeader {
    int status;              // hdt_status_t, first error wins
    int err_pos;             // element / sequence where it was detected
    long long nnz;           // unmasked pairs
    long long visited;       // sum over blocks of rows x span
    StageDesc st[HDT_MAX_STAGES + 1];
    int tail;                // always 0 on the device: the last word of the header to arrive on the host
};

// Host-side pointers to one stage's arrays inside the workspace.
struct StagePtrs {
    int *tok, *par, *rng, *up, *scu, *blocks, *queue, *queue_split;
};

}  // namespace hdt

struct hdt_index {
    int batch, total_tokens, block_m, block_m_upper, n_stages;
    int directions;   // bits 1 | 2 | 4: child->parent, sibling<->sibling, parent->child entries kept (7 = full rule)
    long long nnz, visited;
    hdt::StageDesc desc[HDT_MAX_STAGES + 1];
    hdt::StagePtrs st[HDT_MAX_STAGES];
    void *workspace;
    size_t workspace_bytes;
    const int *rank;                  // device [total_tokens]: a token's number among its siblings (undefined for roots and PAD)
    // Deferred build: the device header is on its way to h_pinned; hdt::index_ready() waits for it
    // and fills n_stages, nnz, visited and desc.
    int pending;                      // 1 until the header has been read
    int failed;                       // hdt_status_t found in the header (or by its check), 0 = fine
    int err_pos, max_stages;
    hdt::DevHeader *h_pinned;         // pinned landing buffer (from a pool), nullptr once released
    cudaEvent_t hdr_ev;               // recorded behind the copy of the header into h_pinned
    const hdt::DevHeader *hdr_dev;    // the header in the index workspace
    cudaStream_t stream;              // stream of the build
};

namespace hdt {

int set_error(int code, const char *fmt, ...);
// Waits (if the build was deferred) until the counts of the index are on the host; returns the
// structure error of the build, if any.
int index_ready(const hdt_index *ix);
int *device_status_ptr();  // device address of the failure word kernels report into
extern std::atomic<long long> g_launches;
inline void count_launch(int n = 1) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// Optional per-kernel timing with CUDA events on the launch stream (off by default).
enum ProfId { PROF_INDEX = 0, PROF_FWD_STAGE0, PROF_FWD_UPPER, PROF_DELTA, PROF_BWD_STAGE0, PROF_BWD_UPPER,
              PROF_COUNT };
struct ProfScope {
    int slot;
    cudaStream_t st;
    ProfScope(int id, cudaStream_t st, bool enabled = true);
    ~ProfScope();
};

#define HDT_CUDA_CHECK(expr)                                                                  \
    do {                                                                                      \
        cudaError_t e_ = (expr);                                                              \
        if (e_ != cudaSuccess)                                                                \
            return hdt::set_error(HDT_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_)); \
    } while (0)

// State that is set up once per device (function attributes such as the dynamic shared-memory
// limit belong to a device's copy of the kernel, not to the process): one flag per device ordinal,
// read and set for the current device.  Two host threads that race on the first call both do the
// set-up, which is idempotent.
struct DevOnce {
    std::atomic<bool> f[64];
    static int cur() {
        int d = 0;
        if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= 64) d = 0;
        return d;
    }
    bool done() const { return f[cur()].load(std::memory_order_acquire); }
    void set() { f[cur()].store(true, std::memory_order_release); }
};
// Number of SMs of the current device (cached per device ordinal).
int sm_count(int *n_sm);

// Side stream (one per host thread and device, created on first use): work that does not depend
// on the main kernel of a call runs beside it.  fork / join are events for the two hand-overs.
struct Side {
    cudaStream_t s, s2, s3;
    cudaEvent_t fork, join, join2, join3, fork0, join0;      // fork0 / join0: a hand-over of their own for work that starts before `fork`
    cudaEvent_t stage_ev[2 * HDT_MAX_STAGES];                // index build with a kernel chain per stage: [2 s] the stage's compaction is queued, [2 s + 1] its walk
    bool ready;
};
int get_side(Side **out);
extern int g_no_overlap;   // option "no_overlap"
extern int g_force_simt;   // option "force_simt"
extern int g_no_graph;     // option "no_graph"
extern int g_phase_stamps; // option "phase_stamps": the transposed backward runs its instrumented instantiation
extern int g_no_fwd_mc;    // option "no_fwd_mc": blocks that are not self-contained stay on the 128-thread general forward kernel

// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute may
// be scheduled while the kernel before it on the stream still runs (once every CTA of that kernel
// has called pdl_launch_dependents or has exited); pdl_wait then blocks until that kernel has
// completed and its writes are visible.  Both are no-ops in a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
extern int g_no_pdl;       // option "no_pdl"
extern int g_bwd_walk;     // option "bwd_walk": families longer than a row block in the head_dim 64 backward: 0 = one walk on the
                           // warp-specialised kernel, 1 = two walks (no dQ buffer, deterministic), 2 = one walk on the lockstep kernel

// Direction bits inside a row range (paper, "Mathematical Reasoning Tasks": the ListOps attention
// patterns).  Row e of a stage has the key range [lo, hi).  If the range starts at or after e, e is
// the head of the family and the keys after it are its children; otherwise lo is e's parent and
// the other keys are its siblings.  dirs: 1 = child -> parent, 2 = sibling <-> sibling,
// 4 = parent -> child entries are kept; the diagonal always is.
__host__ __device__ __forceinline__ bool dir_ok(int e, int j, int lo, int dirs) {
    if (j == e) return true;
    if (lo >= e) return (dirs & 4) != 0;
    return (dirs & (j == lo ? 1 : 2)) != 0;
}
// The same entry seen from the key: key element `key` has the range [lo, hi), query i lies in it.
__host__ __device__ __forceinline__ bool dir_ok_key(int key, int i, int lo, int dirs) {
    if (i == key) return true;
    if (lo >= key) return (dirs & 1) != 0;            // i is a child of the head `key`
    return (dirs & (i == lo ? 4 : 2)) != 0;           // i is key's parent, or a sibling
}

// Tensor-core kernels: bit j of the result says that column s0 + j (j < W <= 32) of a row's tile is
// one of its kept entries: inside the row's range [jl, jh) (tile-relative) and, with direction
// bits (DIRS), not switched off.  c_self / c_head: tile-relative columns of the row itself and of
// its parent (far negative for a head row); keep_head / keep_rest: whether the parent entry / every
// other entry of the range is kept (see dir_ok).
template <bool DIRS>
__device__ __forceinline__ uint32_t keep_mask(int s0, int W, int jl, int jh, int c_self, int c_head, bool keep_head,
                                              bool keep_rest) {
    const int lo = max(jl - s0, 0), hi = min(jh - s0, W);
    if (hi <= lo) return 0u;
    uint32_t m = (hi >= 32 ? 0xffffffffu : ((1u << hi) - 1u)) & ~((1u << lo) - 1u);
    if constexpr (DIRS) {
        uint32_t k = keep_rest ? 0xffffffffu : 0u;
        const int cs = c_self - s0, ch = c_head - s0;
        if (cs >= 0 && cs < 32) k |= 1u << cs;
        if (ch >= 0 && ch < 32) k = keep_head ? (k | (1u << ch)) : (k & ~(1u << ch));
        m &= k;
    }
    return m;
}

// SIMT attention launchers (hdt_attn_simt.cu).  One launch handles one stage.
struct FwdStageArgs {
    // stage view
    int n, nb, H;
    const int *tok;     // nullptr: identity (stage 0)
    const int *rng, *up, *blocks, *queue;
    const int *queue_split;  // SELF non-EMPTY blocks first (n_fused of them), then the rest
    int n_fused;
    const void *q, *k, *v;
    float scale_log2;   // softmax_scale * log2(e)
    // Stages run bottom-up.  carry_*: partial results the stages below left for this stage's
    // elements, indexed by element ([n, H, D] and [n, H]); nullptr for stage 0.
    const float *carry_o, *carry_lse;
    // Every stage writes its merged result to the caller's tensors (later stages overwrite the
    // rows they complete) ...
    void *o;            // dtype [T,H,D]
    float *lse;         // [H,T]
    int T;
    // ... and, for elements that live on in the next stage, to that stage's buffers at up[e]
    // ([n_next, H, D] and [n_next, H]); nullptr for the last stage.
    float *part_o, *part_lse;
    // own_*: when set, the kernel only writes its own partial result per element ([n,H,D], [n,H])
    // and does no merging or final write (the stage runs beside stage 0; merge_fwd finishes it)
    float *own_o, *own_lse;
    int *status;        // device failure word
    int rest_only;      // general kernel: only blocks after the first n_fused
    int no_persistent;  // option: do not use the persistent kernels
    int block_rows;     // max rows of a block in this stage
    int dirs;           // direction bits kept (7 = full rule), see dir_ok
    const int *tok_rows;  // SIMT kernels: token map of the block rows (nullptr: identity); `tok` maps the keys
    int part;             // launch_fwd_tc: 0 = all blocks, 1 = only the self-contained ones (looping kernel), 2 = only the others
    // Gathering kernel, stage 1 run after stage 0 (final_merge = 1): instead of leaving its own
    // partial result it completes every element of the stage: its own result, stage 0's partial
    // (carry_*) and, for elements that live on in stage 2, that stage's own partial (next_own_*,
    // at up[e]; nullptr without a stage 2) are merged and written to o / lse at the element's token.
    // final_merge = 2: the stage's own result is the element's result (nothing to merge; cross-attention):
    // bf16 rows and LSE straight to the element's token, no partial buffers.
    int final_merge;
    const float *next_own_o, *next_own_lse;
    const DevHeader *hdr; // set: the index build is still in flight; the looping kernel reads n_fused and stage 1's size here
    size_t ws_bytes;      // with hdr: bytes behind part_o (the caller's workspace)
    int n_empty;          // EMPTY blocks of the stage (0 where the caller does not know): when they are all that is left
                          // beside the self-contained blocks, a kernel without shared memory and TMEM writes their rows
};

struct BwdStageArgs {
    int n, nb, H, T;
    const int *tok;
    const int *rng, *up, *blocks, *queue;
    const int *queue_split;
    int n_fused;
    const void *q, *k, *v, *d_o;
    const float *lse;    // [H,T] final
    const float *delta;  // [H,T]; nullptr: the kernels compute dO . O of their rows themselves (needs o)
    const void *o;       // forward output, dtype [T,H,D]; read only when delta is nullptr
    float scale, scale_log2;
    const float *carry_dq, *carry_dk, *carry_dv;  // [n,H,D] partials from the stages below, or nullptr
    void *dq, *dk, *dv;                           // dtype [T,H,D], written by every stage
    float *part_dq, *part_dk, *part_dv;           // [n_next,H,D] next stage's buffers (at up[e]), or nullptr
    float *own_dq, *own_dk, *own_dv;              // when set: own gradients only, [n,H,D] (see FwdStageArgs)
    int *status;                                  // device failure word
    int rest_only;                                // general kernel: only blocks after the first n_fused
    int no_persistent;                            // option: do not use the persistent kernels
    int block_rows;                               // max rows of a block in this stage
    int dirs;                                     // direction bits kept (7 = full rule), see dir_ok
    const int *tok_rows;                          // SIMT kernel: token map of the block rows (nullptr: identity); `tok` maps the walked span
    int phases;                                   // 0 = both, 1 = rows as queries only (dQ), 2 = rows as keys only (dK, dV); SIMT and gathering kernels
    // Gathering kernel, stage 1 run after stage 0 (final_merge = 1): the element's gradients are its
    // own plus stage 0's partials (carry_*) plus, for elements that live on in stage 2, that stage's
    // own (next_own_*, at up[e]; nullptr without a stage 2); they go to dq / dk / dv at its token.
    // final_merge = 2: the element's own gradients alone, straight to its token's rows (cross-attention;
    // with phases = 1 only dq, with phases = 2 only dk and dv are written).
    int final_merge;
    const float *next_own_dq, *next_own_dk, *next_own_dv;
    float *dq_acc;                                // stage 0, head_dim 64: fp32 [T,H,64] buffer, zero on entry, that the one-walk kernel of the
                                                  // split families adds its dQ tiles to (nullptr: they are walked twice instead)
    int n_empty;                                  // EMPTY blocks of the stage (-1: unknown)
    void *self_stream;                            // stage 0 with dq_acc: stream (cudaStream_t, already forked from the caller's) for the kernel of the
                                                  // self-contained blocks, which then runs beside the one-walk kernel of the others (nullptr: behind it)
    int gather_end_q, gather_end_k;               // gathering kernel: elements at or beyond these read as zero rows on the Q/dO and the K/V side (0: n)
};

// The stages above 0 of a deep tree in own-partial mode, all in one launch of the SIMT kernels: what differs
// from stage to stage, and where the stage's CTAs start in the launch's grid.
struct MultiStage {
    int n, nb, cum;
    const int *tok, *rng, *up, *blocks, *queue;
    float *own[3];       // forward: own[0] = O; backward: dQ, dK, dV
    float *own_lse;      // forward only
};
struct MultiFwdArgs { FwdStageArgs base; int n; MultiStage st[HDT_MAX_STAGES - 1]; };
struct MultiBwdArgs { BwdStageArgs base; int n; MultiStage st[HDT_MAX_STAGES - 1]; };
int launch_fwd_simt_multi(const MultiFwdArgs &m, int head_dim, int dtype, cudaStream_t st);
int launch_bwd_simt_multi(const MultiBwdArgs &m, int head_dim, int dtype, cudaStream_t st);
int launch_fwd_simt(const FwdStageArgs &a, int head_dim, int dtype, cudaStream_t st);
// Tensor-core (TMA + tcgen05) stage-0 kernels for bf16 (hdt_attn_tc.cu).
int launch_fwd_tc(const FwdStageArgs &a, int head_dim, cudaStream_t st);
int launch_bwd_tc(const BwdStageArgs &a, int head_dim, cudaStream_t st);
// Stages above 0 in own-partial mode on the tensor-core kernels (rows gathered through tok).
int launch_fwd_tc_upper(const FwdStageArgs &a, int head_dim, cudaStream_t st);
int launch_bwd_tc_upper(const BwdStageArgs &a, int head_dim, cudaStream_t st);
int read_bwd_phase_cycles(long long *out16);
int read_bwd_w_marks(long long *out128);
int read_bwd_w_tiles(long long *out512);          // the warp-specialised one-walk backward: see hdt_debug_bwd_w_cycles
int read_bwd_t_phase_cycles(long long *out16);   // adds to out16
int read_bwd_t_timeline(long long *out2048);     // per CTA of the last instrumented launch: entry, first tiles in, end (ns), SM
int read_fwd_phase_cycles(long long *out16);
int read_fwd_timeline(long long *out4096);       // per CTA of the last instrumented looping forward: entry, first tiles in, end (ns), SM
int launch_bwd_simt(const BwdStageArgs &a, int head_dim, int dtype, cudaStream_t st);
int launch_delta(const void *o, const void *d_o, float *delta, int T, int H, int head_dim, int dtype,
                 cudaStream_t st);
// One launch that completes every token of stage 1 (= every token that lives in a stage above 0):
// stage 0's partial merged with the own partials of all upper stages the token belongs to, found
// by following the `up` maps.  nt = 1 tensor (forward: O with LSE) or 3 (backward: dQ, dK, dV).
struct ChainArgs {
    int n1, H, T, n_stages, nt;
    const int *tok1;
    const int *up[HDT_MAX_STAGES];           // up[s]: stage s -> stage s+1
    const float *own[HDT_MAX_STAGES][3];     // own[s][t], s >= 1
    const float *own_lse[HDT_MAX_STAGES];    // forward only
    const float *base[3];                    // stage 0's partials for stage 1's elements
    const float *base_lse;
    void *out[3];
    float *lse;
};
int launch_chain_merge(const ChainArgs &c, int head_dim, int dtype, cudaStream_t st);

}  // namespace hdt
