// Test hook for the sm_100a primitives: one CTA computes C[128 x N] = A * B with bf16 operands
// staged by TMA into 128-byte-swizzled shared memory and multiplied by tcgen05.mma, for every
// combination of K-major / MN-major operands the attention kernels use.  Checked against a
// plain matmul in tests/test_gpu_primitives.py.
#include "hdt_internal.cuh"
#include "hdt_sm100.cuh"
#include "hdt_tmap.cuh"

namespace hdt {
using namespace sm100;

struct DebugGemmArgs {
    int N, K, a_mn, b_mn;
    float *c;  // [128, N]
    int *status;
};

__global__ void __launch_bounds__(128) k_debug_gemm(const __grid_constant__ CUtensorMap tm_a,
                                                    const __grid_constant__ CUtensorMap tm_b, const DebugGemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sA = sm, *sB = sm + 2 * 16384;
    uint64_t *bar = (uint64_t *)(sm + 4 * 16384);
    uint32_t *slot = (uint32_t *)(bar + 2);
    volatile int *abort_flag = (volatile int *)(slot + 1);
    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid == 0) {
        mbar_init(&bar[0], 1);
        mbar_init(&bar[1], 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) tmem_alloc(slot, 128);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *slot;
    if (tid == 0) {
        mbar_expect_tx(&bar[0], 4 * 16384);
        // two 64-column sub-tiles of each operand: box (64, 1, 128) at column 64 s, row 0
        for (int s = 0; s < 2; ++s) {
            tma_load_3d(sA + s * 16384, &tm_a, 64 * s, 0, 0, &bar[0]);
            tma_load_3d(sB + s * 16384, &tm_b, 64 * s, 0, 0, &bar[0]);
        }
    }
    bool ok = mbar_wait(&bar[0], 0, abort_flag, 400000000LL);
    if (tid == 0 && ok) {
        tc_fence_after();
        const uint32_t idesc = idesc_bf16(g.N, g.a_mn != 0, g.b_mn != 0);
        for (int kk = 0; kk < g.K / 16; ++kk) {
            const uint64_t da = g.a_mn ? smem_desc(smem_u32(sA) + kk * 2048, 16384, 1024)
                                       : smem_desc(smem_u32(sA) + (kk / 4) * 16384 + (kk % 4) * 32, 0, 1024);
            const uint64_t db = g.b_mn ? smem_desc(smem_u32(sB) + kk * 2048, 16384, 1024)
                                       : smem_desc(smem_u32(sB) + (kk / 4) * 16384 + (kk % 4) * 32, 0, 1024);
            mma_ss(tmem, da, db, idesc, kk > 0);
        }
        mma_commit(&bar[1]);
    }
    ok = ok && mbar_wait(&bar[1], 0, abort_flag, 400000000LL);
    tc_fence_after();
    if (!ok && tid == 0) atomicCAS(g.status, 0, HDT_ERR_TIMEOUT);
    for (int c0 = 0; c0 < g.N; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + c0, r);
        tmem_wait_ld();
        for (int j = 0; j < 32; ++j)
            if (c0 + j < g.N) g.c[(size_t)tid * g.N + c0 + j] = __uint_as_float(r[j]);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 128);
}

}  // namespace hdt

using namespace hdt;

// a: bf16 [128, K] (a_mn = 0) or [K, 128] (a_mn = 1); b: bf16 [N, K] (b_mn = 0) or [K, N] (b_mn = 1);
// c: float [128, N].  N, K multiples of 16, <= 128.  Test hook; waits for the result.
extern "C" int hdt_debug_gemm(const void *a, const void *b, float *c, int32_t N, int32_t K, int32_t a_mn,
                              int32_t b_mn, void *stream) {
    if (!a || !b || !c || N < 16 || N > 128 || N % 16 || K < 16 || K > 128 || K % 16)
        return set_error(HDT_ERR_INVALID_ARG, "hdt_debug_gemm: bad arguments");
    cudaStream_t st = (cudaStream_t)stream;
    CUtensorMap ta, tb;
    // tensors as [rows, 1, cols]
    int rc = make_tmap_bf16(&ta, a, a_mn ? 128 : K, 1, a_mn ? K : 128, 128);
    if (rc) return rc;
    rc = make_tmap_bf16(&tb, b, b_mn ? N : K, 1, b_mn ? K : N, 128);
    if (rc) return rc;
    int *status = device_status_ptr();
    if (!status) return HDT_ERR_CUDA;
    DebugGemmArgs g{N, K, a_mn, b_mn, c, status};
    const int smem = 4 * 16384 + 1024 + 64;
    HDT_CUDA_CHECK(cudaFuncSetAttribute(k_debug_gemm, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    k_debug_gemm<<<1, 128, smem, st>>>(ta, tb, g);
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    return hdt_device_status(stream);
}


namespace hdt {
// One CTA that sets up what the attention kernels set up (an mbarrier, TMEM columns) and then waits on
// a barrier nobody ever arrives on: no TMA copy and no MMA is issued, so nothing is in flight when the
// bounded wait gives up.  It then takes the failure path of the attention kernels: abort flag,
// HDT_ERR_TIMEOUT with kernel id 15 / wait site 1 / the wait limit's low bits in the status word, TMEM
// released, normal exit.  second[0] counts the threads that saw the abort flag and left their own wait early.
__global__ void __launch_bounds__(128) k_debug_wait(long long limit_cycles, int *status, int *second) {
    __shared__ uint64_t bar;
    __shared__ uint32_t slot;
    __shared__ int abort_flag_s;
    volatile int *abort_flag = &abort_flag_s;
    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid == 0) {
        mbar_init(&bar, 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 0) tmem_alloc(&slot, 32);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = slot;
    const long long t0 = clock64();
    const bool ok = mbar_wait(&bar, 0, abort_flag, limit_cycles);
    if (!ok) {
        if (clock64() - t0 <= limit_cycles) atomicAdd(second, 1);       // left early through the abort flag
        if (tid == 0) {
            if (atomicCAS(status, 0, HDT_ERR_TIMEOUT) == 0) {
                status[1] = (15 << 8) | 1;
                status[2] = (int)(limit_cycles & 0x7fffffff);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 32);
}
}  // namespace hdt

// Test hook for the failure path of the bounded device-side waits (no counterpart in the paper): see
// k_debug_wait.  Returns what hdt_device_status returns afterwards (HDT_ERR_TIMEOUT when the path
// works) and, in *left_early, how many of the 128 threads stopped waiting because of the abort flag.
extern "C" int hdt_debug_wait_timeout(int64_t limit_cycles, int32_t *left_early, void *stream) {
    if (limit_cycles < 1000 || limit_cycles > 2000000000LL)
        return set_error(HDT_ERR_INVALID_ARG, "hdt_debug_wait_timeout: limit_cycles must be 1e3..2e9");
    cudaStream_t st = (cudaStream_t)stream;
    int *status = device_status_ptr();
    if (!status) return HDT_ERR_CUDA;
    k_debug_wait<<<1, 128, 0, st>>>((long long)limit_cycles, status, status + 3);
    count_launch();
    HDT_CUDA_CHECK(cudaGetLastError());
    HDT_CUDA_CHECK(cudaStreamSynchronize(st));
    int h[4] = {0, 0, 0, 0};
    HDT_CUDA_CHECK(cudaMemcpy(h, status, sizeof(h), cudaMemcpyDeviceToHost));
    if (left_early) *left_early = h[3];
    return hdt_device_status(stream);
}

// Diagnostics (no counterpart in the paper): SM cycles that CTA 0 of the persistent backward kernel
// spent in each of its phases since the last call (out16[0..11]) and the items it processed (out16[12]).
// Waits for the device.
extern "C" int hdt_debug_fwd_phase_cycles(int64_t *out16) {
    if (!out16) return set_error(HDT_ERR_INVALID_ARG, "hdt_debug_fwd_phase_cycles: null pointer");
    HDT_CUDA_CHECK(cudaDeviceSynchronize());
    return read_fwd_phase_cycles((long long *)out16);
}

extern "C" int hdt_debug_bwd_phase_cycles(int64_t *out16) {
    if (!out16) return set_error(HDT_ERR_INVALID_ARG, "hdt_debug_bwd_phase_cycles: null pointer");
    HDT_CUDA_CHECK(cudaDeviceSynchronize());
    const int rc = read_bwd_phase_cycles((long long *)out16);
    return rc ? rc : read_bwd_t_phase_cycles((long long *)out16);
}

// Diagnostics: per CTA (up to 512) of the last instrumented transposed backward launch (option
// "phase_stamps"): global timer at entry, when the first input tiles had arrived, at the end of its
// item loop (ns), and the SM it ran on.  Waits for the device.
extern "C" int hdt_debug_bwd_timeline(int64_t *out2048) {
    if (!out2048) return hdt::set_error(HDT_ERR_INVALID_ARG, "hdt_debug_bwd_timeline: null pointer");
    HDT_CUDA_CHECK(cudaDeviceSynchronize());
    return hdt::read_bwd_t_timeline((long long *)out2048);
}

// The same for the looping forward (up to 1024 CTAs).
extern "C" int hdt_debug_fwd_timeline(int64_t *out4096) {
    if (!out4096) return hdt::set_error(HDT_ERR_INVALID_ARG, "hdt_debug_fwd_timeline: null pointer");
    HDT_CUDA_CHECK(cudaDeviceSynchronize());
    return hdt::read_fwd_timeline((long long *)out4096);
}
