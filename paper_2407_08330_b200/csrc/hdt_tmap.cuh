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

// base: device pointer, 16-byte aligned; D: inner extent (elements, D * 2 bytes a multiple of 16).
inline int make_tmap_bf16(CUtensorMap *tm, const void *base, int D, int H, long long T, int box_rows) {
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
