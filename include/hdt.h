/*
 * libhdt — hierarchical sparse attention of the Hierarchical Document Transformer (HDT)
 * for NVIDIA B200 (sm_100a).  C ABI; no C++ or framework types cross this boundary.
 *
 * The operation (paper, section "Hierarchical Document Transformer", paragraph
 * "Hierarchical Attention", and Algorithm 1 in the appendix): tokens are laid out in document
 * order with anchor tokens ([DOC], one [SEC] per section, one [SENT] per sentence).  Every
 * token attends to its parent, its siblings (same parent, itself included) and its children;
 * all other query-key pairs are masked with -inf before the row softmax:
 *
 *     A = Q K^T * softmax_scale,   S = softmax(A masked),   O = S V,
 *     LSE_i = log sum_{j unmasked} exp(A_ij).
 *
 * The mask is the same for all heads and differs per sequence.
 *
 * Calling sequence:  hdt_build_index  (once per batch of documents; the index is valid for all
 * layers, heads, forward and backward)  ->  hdt_attn_fwd / hdt_attn_bwd  (any number of times)
 * ->  hdt_index_destroy.
 *
 * Conventions
 *  - "device" pointers are CUDA device memory of the current device, owned by the caller.
 *    The library never allocates or frees device memory; scratch comes in caller workspaces.
 *  - Q, K, V, O, dO, dQ, dK, dV: packed token-major [total_tokens, heads, head_dim],
 *    contiguous, 16-byte aligned, element type given by hdt_dtype_t.
 *    LSE: float [heads, total_tokens], natural logarithm, softmax_scale included.
 *  - Structure: level[i] in {0 root/[DOC], 1 [SEC], 2 [SENT], 3 regular token, deeper levels
 *    allowed, -1 PAD}; parent[i] = index of the parent token relative to the start of its own
 *    sequence, -1 for the root and for PAD; cu_seqlens[batch+1] cumulative sequence offsets
 *    (cu_seqlens[0] = 0, cu_seqlens[batch] = total_tokens).  Preconditions, checked on the
 *    device by hdt_build_index: the first token of a sequence is its only root (level 0);
 *    0 <= parent[i] < i (sequence-relative); level[i] = level[parent[i]] + 1; tokens are in
 *    document (pre-)order, i.e. a node whose children are all childless is directly followed
 *    by those children; PAD only as a suffix of a sequence.
 *    PAD rows produce O = 0, LSE = -inf and zero gradients.  The Q, K, V and dO rows of PAD tokens
 *    must hold finite numbers: the tensor-core kernels load them with their tile and multiply them
 *    by exact zeros, and 0 x NaN or 0 x inf would reach real rows of the same tile (zero-fill them,
 *    as a padded batch normally is; nothing checks this).
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  hdt_attn_fwd/bwd are
 *    asynchronous on it.  hdt_build_index enqueues its kernels on it and then waits for them,
 *    because it returns the sizes the attention calls need.
 *  - Every function returns an hdt_status_t (HDT_OK = 0, errors negative); nothing throws,
 *    aborts or traps the device.  hdt_last_error() gives a thread-local message.
 */
#ifndef HDT_H_
#define HDT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    HDT_OK = 0,
    HDT_ERR_INVALID_ARG = -1,   /* null pointer, negative size, misaligned buffer            */
    HDT_ERR_BAD_HIERARCHY = -2, /* structure arrays violate a precondition                    */
    HDT_ERR_UNSUPPORTED = -3,   /* head_dim / dtype / size outside what the kernels cover     */
    HDT_ERR_WORKSPACE = -4,     /* workspace too small                                        */
    HDT_ERR_CUDA = -5,          /* a CUDA runtime call failed; see hdt_last_error()           */
    HDT_ERR_TIMEOUT = -6        /* a bounded device-side wait ran out                         */
} hdt_status_t;

typedef enum { HDT_F32 = 0, HDT_BF16 = 1 } hdt_dtype_t;

#define HDT_MAX_STAGES 24

typedef struct {
    int32_t block_m;    /* max rows per row block, 1..128; 0 = default 128                     */
    int32_t max_stages; /* max hierarchy height handled, 1..HDT_MAX_STAGES; 0 = default 4
                           ([DOC]/[SEC]/[SENT]/token documents need 3)                        */
    int32_t block_m_upper; /* max rows per row block in the stages above 0, 1..128; 0 = default
                           128 (whole families per block for the tensor-core kernels; the fp32
                           SIMT kernels of those stages get more CTAs from smaller blocks)    */
    int32_t mask_off;   /* directed variants of the rule (paper, "Mathematical Reasoning Tasks": the
                           ListOps attention patterns): bit 0 switches OFF a token attending to its
                           parent, bit 1 to its other siblings, bit 2 to its children; the diagonal
                           always stays.  0 = the full parent/sibling/child rule.  The family
                           ranges of the index do not change; nnz counts the remaining pairs and
                           the attention kernels drop the switched-off entries inside each range */
    int32_t deferred;   /* 0: hdt_build_index waits until the index is complete and reports structure
                           errors itself.  1: it returns as soon as the work is queued on the stream;
                           the first call that needs the counts of the index on the host
                           (hdt_index_info, hdt_index_export, the workspace queries, the attention and
                           positional-encoding calls) waits instead and returns the structure error,
                           if any; every later call on that index returns it too.  hdt_attn_fwd on a
                           bf16 index still in flight queues its stage-0 kernel first (the kernel
                           reads the counts on the device) and waits only then.  The structure
                           arrays and the workspace must stay allocated until the stream has
                           passed the build (as for any asynchronous call)                      */
    int32_t reserved[3];
} hdt_index_params_t;

typedef struct hdt_index hdt_index_t; /* opaque host object; views into the caller's workspace */

/*
 * One stage of the index, device pointers into the index workspace (read-only).
 * The index decomposes the mask into "families" {node} + its children, each of which is a
 * contiguous range of a compacted token array; stage s handles the families whose members are
 * all childless after the children handled by stages < s have been removed.  This replaces the
 * per-tile emptiness test and the level sort of keys of the paper's Algorithm 1 (the "sort K, V"
 * and "compute mask / if non-zero" steps): a row block's non-empty tiles are exactly its key
 * span [a, b).
 */
typedef struct {
    int32_t n;               /* elements in this stage's array                                */
    int32_t n_blocks;        /* row blocks                                                    */
    const int32_t *tok;      /* [n]   global token id of element e                            */
    const int32_t *par;      /* [n]   index in this array of e's parent, -1 root / PAD        */
    const int32_t *rng;      /* [n,2] key range [lo,hi) of row e in this array; (0,0) = none  */
    const int32_t *up;       /* [n]   index of e in the next stage's array, -1 if removed     */
    const int32_t *scu;      /* [batch+1] sequence offsets in this array                      */
    const int32_t *blocks;   /* [n_blocks,5] r0, r1, a, b, flags (HDT_BLK_*)                  */
    const int32_t *queue;    /* [n_blocks] block ids, cost (r1-r0)*(b-a) descending, id asc.  */
    const int32_t *queue_split; /* [n_blocks] the same order inside two groups: first the n_fused
                                blocks that are SELF and not EMPTY, then all others             */
    int32_t n_fused;
} hdt_stage_view_t;

#define HDT_BLK_SELF 1  /* key span inside the row block                                      */
#define HDT_BLK_DENSE 2 /* every row's range equals the span: no in-tile masking needed       */
#define HDT_BLK_CARRY 4 /* some row also has a partial result from a later stage              */
#define HDT_BLK_EMPTY 8 /* no row has a key in this stage                                     */

/*
 * Bytes of device workspace hdt_build_index needs (host computation, no CUDA call).
 * Returns 0 for invalid arguments.
 */
size_t hdt_index_workspace_bytes(int32_t batch, int32_t total_tokens,
                                 const hdt_index_params_t *params /* NULL = defaults */);

/*
 * Build the index of one batch on the device (Algorithm 1's mask test and key ordering, done
 * once per batch instead of per tile and per call).
 *   level      device int8  [total_tokens]
 *   parent     device int32 [total_tokens]
 *   cu_seqlens device int32 [batch+1]
 *   workspace  device, >= hdt_index_workspace_bytes(...), 256-byte aligned; must stay allocated
 *              and untouched until hdt_index_destroy
 *   out        receives a host object (free with hdt_index_destroy)
 * Waits for the stream before returning (unless params->deferred is set: see there).  Errors:
 * HDT_ERR_BAD_HIERARCHY when a precondition on the structure arrays fails or the hierarchy needs
 * more than max_stages stages (no index is returned; a deferred build returns the index and the
 * error comes from the first call that uses it), HDT_ERR_WORKSPACE, HDT_ERR_INVALID_ARG,
 * HDT_ERR_CUDA.
 */
int hdt_build_index(const int8_t *level, const int32_t *parent, const int32_t *cu_seqlens,
                    int32_t batch, int32_t total_tokens, const hdt_index_params_t *params,
                    void *workspace, size_t workspace_bytes, void *stream, hdt_index_t **out);

/* Totals of a built index: stages, unmasked pairs per head, visited pairs (sum of block rows x span). */
int hdt_index_info(const hdt_index_t *index, int32_t *n_stages, int64_t *nnz_pairs,
                   int64_t *visited_pairs);

/* Device views of stage `stage` (0 <= stage < n_stages) for inspection and parity tests. */
int hdt_index_export(const hdt_index_t *index, int32_t stage, hdt_stage_view_t *view);

/* Frees the host object only. */
int hdt_index_destroy(hdt_index_t *index);

/*
 * Bytes of device workspace for hdt_attn_fwd (bwd = 0) or hdt_attn_bwd (bwd = 1) with this
 * index: partial results of the stages above stage 0, and delta = rowsum(dO o O) for backward.
 */
size_t hdt_attn_workspace_bytes(const hdt_index_t *index, int32_t heads, int32_t head_dim,
                                int32_t dtype, int32_t bwd);

/*
 * Forward pass (hierarchical attention equation; Algorithm 1 without its per-tile HBM
 * round trips): O and LSE for every token and head.
 *   q, k, v   device [total_tokens, heads, head_dim] of `dtype`
 *   o         device, same shape and dtype (written)
 *   lse       device float [heads, total_tokens] (written)
 *   softmax_scale <= 0 selects 1/sqrt(head_dim)
 *   workspace device, >= hdt_attn_workspace_bytes(index, heads, head_dim, dtype, 0), 256-byte
 *             aligned; contents are scratch
 * head_dim must be 64 or 128.  Asynchronous on `stream`.
 */
int hdt_attn_fwd(const hdt_index_t *index, const void *q, const void *k, const void *v, void *o,
                 float *lse, int32_t heads, int32_t head_dim, int32_t dtype, float softmax_scale,
                 void *workspace, size_t workspace_bytes, void *stream);

/*
 * Backward pass.  The paper prints no backward; this is the derivative of the forward map:
 *   delta_i = sum_c dO_ic O_ic;  P_ij = exp(A_ij - LSE_i);  dV = P^T dO;  dP = dO V^T;
 *   dS = P o (dP - delta);  dQ = scale dS K;  dK = scale dS^T Q        (unmasked pairs only).
 *   o, lse    the forward results for the same q, k, v
 *   d_o       device, gradient of the loss w.r.t. O
 *   dq, dk, dv device, written (same shape and dtype as q)
 *   workspace device, >= hdt_attn_workspace_bytes(..., 1), 256-byte aligned
 * Asynchronous on `stream`.
 */
int hdt_attn_bwd(const hdt_index_t *index, const void *q, const void *k, const void *v,
                 const void *o, const float *lse, const void *d_o, void *dq, void *dk, void *dv,
                 int32_t heads, int32_t head_dim, int32_t dtype, float softmax_scale,
                 void *workspace, size_t workspace_bytes, void *stream);

/* Thread-local text of the last error returned on this thread ("" if none). */
const char *hdt_last_error(void);

/* Number of kernel launches the library has issued in this process (for benchmarks). */
int64_t hdt_launch_count(void);

/*
 * Optional per-kernel timing for benchmarks (no counterpart in the paper).  When enabled, the
 * library brackets its launches with CUDA events on the launch stream.  Kernel ids:
 * 0 index build (all its kernels), 1 forward stage 0, 2 forward upper stages, 3 delta,
 * 4 backward stage 0, 5 backward upper stages.  hdt_profile_read waits for the recorded events,
 * returns the number of bracketed launches and their summed device time in milliseconds since
 * the last reset, and clears them when reset != 0.
 */
int hdt_profile_enable(int32_t on);
const char *hdt_profile_name(int32_t id);
int hdt_profile_read(int32_t id, int64_t *launches, double *total_ms, int32_t reset);

/*
 * Forward pass without a caller workspace (the paper has no counterpart; this is an addition for
 * embedding the library).  Same inputs, outputs and results as hdt_attn_fwd, but the partial
 * results of the upper stages are kept in a fixed array inside the library instead of a
 * workspace.  It is meant for callers that are not allowed to allocate device memory at the point
 * of the call: code running inside a memory pool that has already handed out all of its budget, a
 * plug-in whose host owns every allocation, or a latency-critical loop where cudaMalloc (which
 * synchronises the device) must not appear.  The call itself performs no cudaMalloc, cudaFree or
 * other allocating call.
 *  - Limit: hdt_attn_workspace_bytes(index, heads, head_dim, dtype, 0) must not exceed
 *    hdt_attn_fwd_static_max_bytes() (8 MiB, enough for about 1 000 anchor tokens x 16 heads x
 *    head_dim 64); larger batches get HDT_ERR_WORKSPACE and a message that says so.  The array
 *    occupies that much memory on every GPU that loads the library, until the process exits.
 *  - The first call on each device looks up the array's device address (a CUDA runtime query);
 *    make that first call outside any stream capture.
 *  - All calls share the one array.  It keeps whatever the last call left, which is harmless:
 *    each call overwrites every entry before reading it, so nothing needs clearing.  Two calls
 *    that overlap on the GPU (different streams, or different threads) race on it and corrupt
 *    each other's results: serialise them.
 * The structure arrays and the index still come from hdt_build_index and its workspace.
 */
size_t hdt_attn_fwd_static_max_bytes(void);
int hdt_attn_fwd_static(const hdt_index_t *index, const void *q, const void *k, const void *v, void *o,
                        float *lse, int32_t heads, int32_t head_dim, int32_t dtype, float softmax_scale,
                        void *stream);

/*
 * Hierarchical positional encoding (paper, paragraph "Hierarchical Positional Encoding", the
 * positional-encoding equation): HPE(p, 2k) = sum_l sin(w_k p^l), HPE(p, 2k+1) = sum_l cos(w_k p^l),
 * w_k = 10000^(-2k/d_model), l = 1..n_levels, where p^l is the number (from 1) of the token's
 * level-l ancestor (or of the token itself) among its siblings, and 0 on levels deeper than the
 * token's own.  The root has p = 0 on every level; PAD tokens get 0 (accumulate = 0) or are left
 * unchanged (accumulate = 1).
 *   index              built from the same level / parent / cu_seqlens (the build leaves every
 *                      token's number among its siblings in the index workspace)
 *   x                  device [total_tokens, d_model] of `dtype`; overwritten (accumulate = 0) or
 *                      incremented (accumulate = 1: token embeddings + HPE, as the encoder input)
 *   workspace          device, >= hdt_hpe_workspace_bytes(index, n_levels), 256-byte aligned
 * d_model must be even.  Asynchronous on `stream`.
 */
size_t hdt_hpe_workspace_bytes(const hdt_index_t *index, int32_t n_levels);
int hdt_hpe(const hdt_index_t *index, const int8_t *level, const int32_t *parent, const int32_t *cu_seqlens,
            int32_t n_levels, int32_t d_model, int32_t dtype, int32_t accumulate, void *x, void *workspace,
            size_t workspace_bytes, void *stream);

/*
 * Decoder cross-attention to a level subset of the encoder tokens (paper, paragraph "Results on
 * FacetSum (Encoder-Decoder Models)": the decoder attends only to [SEC] anchors, to [SEC] and [SENT]
 * anchors, or to every token of the encoder output; the decoder's cross-attention sub-layer of the
 * paragraph "Hierarchical Encoder and Decoder Stacks").  For document b the decoder rows
 * cu_seqlens_q[b] .. cu_seqlens_q[b+1] attend to the encoder tokens of the same document whose level
 * l has bit l set in level_mask (PAD, level -1, is never chosen):
 *     O = softmax(Q Ks^T * scale) Vs,   LSE_i = log sum_j exp(A_ij).
 * A decoder row of a document without a chosen token gets O = 0 and LSE = -inf.
 *   level              device int8 [total_tokens]; cu_seqlens_k / cu_seqlens_q device int32 [batch+1]
 *   q, o, d_o, dq      device [total_q, heads, head_dim] of `dtype`, 16-byte aligned
 *   k, v, dk, dv       device [total_tokens, heads, head_dim]; dk, dv are written for every encoder
 *                      row (zero outside the subset)
 *   lse                device float [heads, total_q]
 *   workspace          device, >= hdt_cross_workspace_bytes(batch, total_tokens, total_q, heads,
 *                      head_dim, dtype, bwd), 256-byte aligned; holds the list of chosen tokens and
 *                      their block records, rebuilt by every call (and delta in the backward)
 * head_dim 64 or 128; softmax_scale <= 0 means 1/sqrt(head_dim).  Asynchronous on `stream`, no
 * host wait.  The chosen rows are read in place through the list (no gathered copy of K, V).
 */
size_t hdt_cross_workspace_bytes(int32_t batch, int32_t total_tokens, int32_t total_q, int32_t heads,
                                 int32_t head_dim, int32_t dtype, int32_t bwd);
int hdt_cross_attn_fwd(const int8_t *level, const int32_t *cu_seqlens_k, const int32_t *cu_seqlens_q, int32_t batch,
                       int32_t total_tokens, int32_t total_q, int32_t level_mask, const void *q, const void *k,
                       const void *v, void *o, float *lse, int32_t heads, int32_t head_dim, int32_t dtype,
                       float softmax_scale, void *workspace, size_t workspace_bytes, void *stream);
int hdt_cross_attn_bwd(const int8_t *level, const int32_t *cu_seqlens_k, const int32_t *cu_seqlens_q, int32_t batch,
                       int32_t total_tokens, int32_t total_q, int32_t level_mask, const void *q, const void *k,
                       const void *v, const void *o, const float *lse, const void *d_o, void *dq, void *dk, void *dv,
                       int32_t heads, int32_t head_dim, int32_t dtype, float softmax_scale, void *workspace,
                       size_t workspace_bytes, void *stream);

/*
 * Waits for `stream`, then returns and clears the first failure a kernel of this library
 * recorded on the device: HDT_ERR_TIMEOUT when a bounded wait (on a TMA or tensor-core
 * completion barrier) ran out; results of that call are then undefined.  HDT_OK if none.
 * While a failure is recorded and not yet cleared, every later tensor-core kernel of the library
 * sees it at its start and does nothing (its outputs stay unwritten) although hdt_attn_fwd /
 * hdt_attn_bwd still return HDT_OK, because they do not wait for the device: a caller that needs
 * to know calls this function after the step.  (No counterpart in the paper.)
 */
int hdt_device_status(void *stream);

#ifdef __cplusplus
}
#endif
#endif /* HDT_H_ */
