// Host side: TMA tensor maps for [T, H, D] bf16 tensors (D innermost), box = (64, 1, box_rows),
// 128-byte swizzle.  cuTensorMapEncodeTiled is fetched through the runtime, so libcuda is not
// linked.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "hdt_internal.cuh"

namespace hdt {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// A tensor map is a function of (address, extents, box) only, and a training loop comes back with the
// same tensors step after step: each host thread keeps the maps it made in a small direct-mapped
// table (a call of the attention makes some thirty of them).
struct TmapEntry {
    alignas(64) CUtensorMap map;
    const void *base;
    long long T;
    int D, H, box_rows, kind;      // kind: 1 = bf16 [T, H, D], 2 = fp32 accumulation buffer; 0 = empty
};
inline TmapEntry *tmap_slot(const void *base, int D, int H, long long T, int box_rows, int kind, bool *hit) {
    static thread_local TmapEntry table[128];
    const uintptr_t a = (uintptr_t)base;
    const unsigned h = (unsigned)((a >> 8) * 0x9E3779B1u) ^ ((unsigned)box_rows * 0x85EBCA6Bu) ^ ((unsigned)kind << 5) ^ (unsigned)D;
    TmapEntry *e = &table[(h ^ (h >> 15)) & 127u];
    *hit = e->kind == kind && e->base == base && e->T == T && e->D == D && e->H == H && e->box_rows == box_rows;
    return e;
}

// base: device pointer, 16-byte aligned; D: inner extent (elements, D * 2 bytes a multiple of 16).
inline int make_tmap_bf16(CUtensorMap *tm, const void *base, int D, int H, long long T, int box_rows) {
    bool hit = false;
    TmapEntry *slot = tmap_slot(base, D, H, T, box_rows, 1, &hit);
    if (hit) { *tm = slot->map; return HDT_OK; }
    const int rc = [&]() -> int {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return set_error(HDT_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)(T > 0 ? T : 1)};
    cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)D * 2 * (cuuint64_t)H};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return set_error(HDT_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return HDT_OK;
    }();
    if (rc == HDT_OK) { slot->map = *tm; slot->base = base; slot->T = T; slot->D = D; slot->H = H; slot->box_rows = box_rows; slot->kind = 1; }
    return rc;
}

// fp32 accumulation buffer [T, H, 64] for reduce-add copies: box = (32 floats, 1, box_rows), i.e.
// 128-byte rows with the 128-byte swizzle; a [rows x 64] tile is two such boxes (x = 0 and x = 32).
inline int make_tmap_f32_acc(CUtensorMap *tm, const void *base, int H, long long T, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return set_error(HDT_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[3] = {64, (cuuint64_t)H, (cuuint64_t)(T > 0 ? T : 1)};
    cuuint64_t strides[2] = {64 * 4, 64 * 4 * (cuuint64_t)H};
    cuuint32_t box[3] = {32, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return set_error(HDT_ERR_CUDA, "cuTensorMapEncodeTiled (fp32) failed with CUresult %d", (int)r);
    return HDT_OK;
}

// Output tiles of the persistent backward kernels leave through TMA stores.  A block has 1..128 rows
// and a store box has a fixed number of rows, so each gradient tensor (dq, dk, dv) gets seven maps
// with boxes of 64, 32, ..., 1 rows and a tile is stored as two (possibly overlapping) boxes of the
// largest size that fits.
struct StoreMaps { CUtensorMap m[3][7]; };
struct OutMaps { CUtensorMap m[7]; };     // the same for one tensor (the forward's O)

// Self-contained (SELF, non-EMPTY) blocks of stage 0 at head_dim 64 through the transposed looping
// backward (hdt_attn_tc_bwd_t.cu); the maps are those of q, k, v, dO with boxes of 128 rows.
int launch_bwd_tc_fused64(const BwdStageArgs &a, const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv,
                          const CUtensorMap &tdo, const StoreMaps &outs, cudaStream_t st);

// The blocks after the first n_fused of queue_split (pieces of families longer than a row block, and
// EMPTY blocks) at head_dim 64 through the warp-specialised one-walk backward (hdt_attn_tc_bwd_w.cu):
// dK, dV rows are written, dQ tiles are added to a.dq_acc through `tacc` (the caller converts the sums).
// n_empty: EMPTY blocks among them (-1: unknown).
int launch_bwd_tc_onewalk64(const BwdStageArgs &a, const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv,
                            const CUtensorMap &tdo, const StoreMaps &outs, const CUtensorMap &tacc, int n_empty, cudaStream_t st);

}  // namespace hdt
