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

extern "C" int hdt_debug_bwd_w_tiles(int64_t *out512) {
    if (!out512) return hdt::set_error(HDT_ERR_INVALID_ARG, "hdt_debug_bwd_w_tiles: null pointer");
    HDT_CUDA_CHECK(cudaDeviceSynchronize());
    return hdt::read_bwd_w_tiles((long long *)out512);
}

extern "C" int hdt_debug_bwd_w_marks(int64_t *out128) {
    if (!out128) return hdt::set_error(HDT_ERR_INVALID_ARG, "hdt_debug_bwd_w_marks: null pointer");
    HDT_CUDA_CHECK(cudaDeviceSynchronize());
    return hdt::read_bwd_w_marks((long long *)out128);
}

namespace hdt {
// Timing probe of the tensor pipe: one CTA, one thread issues `reps` groups of `per_group` MMAs
// (M = 128, N = n, K = 16 each, operands = whatever the shared memory / TMEM holds: only the time
// matters), commits once, and the SM clock cycles from the first issue to the completion of the last
// MMA go to out[0], those of the issue loop alone to out[1].  mode bit 0: A from TMEM; bit 1: consecutive
// MMAs alternate between two accumulators, so that none depends on the one before it.
__global__ void __launch_bounds__(128) k_debug_mma_rate(int n, int reps, int per_group, int mode, int b_mn, long long *out) {
    extern __shared__ __align__(1024) uint8_t sm[];
    __shared__ uint64_t bars2[2];
    __shared__ uint32_t slot;
    __shared__ int abort_s;
    volatile int *abort_flag = &abort_s;
    const int tid = threadIdx.x, warp = tid >> 5;
    for (int i = tid; i < 4 * 16384 / 4; i += 128) ((uint32_t *)sm)[i] = 0x3c003c00u;     // finite bf16 values
    if (tid == 0) { mbar_init(&bars2[0], 1); mbar_init(&bars2[1], 1); *abort_flag = 0; fence_mbar_init(); }
    const int n_issuers = (mode & 4) ? 2 : 1;      // mode bit 2: warps 0 and 1 both issue (accumulators 64 columns apart)
    uint64_t &bar = bars2[warp & 1];
    fence_proxy_async_smem();
    if (warp == 0) tmem_alloc(&slot, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = slot;
    if (warp < n_issuers) {
        long long t0 = 0, t1 = 0;
        if (elect_one()) {
            const uint32_t idesc = idesc_bf16(n > 64 && n_issuers == 2 ? 64 : n, false, b_mn != 0);
            const uint64_t da = smem_desc(smem_u32(sm), 0, 1024);
            const uint64_t db = b_mn ? smem_desc(smem_u32(sm) + 2 * 16384, 16384, 1024) : smem_desc(smem_u32(sm) + 2 * 16384, 0, 1024);
            const int alt = (mode >> 1) & 1, at = mode & 1;
            t0 = clock64();
            for (int r = 0; r < reps; ++r) {
                const uint32_t d = tmem + 256u * (r & 1) + 64u * warp;
                for (int g = 0; g < per_group; ++g) {
                    const uint32_t dd = d + (alt ? 128u * (g & 1) : 0u);
                    const uint32_t acc = alt ? (g > 1) : (g > 0);
                    if (at) mma_ts(dd, tmem + 448u + 8u * (g & 3), db + (uint64_t)((g & 3) * (b_mn ? 128 : 2)), idesc, acc);
                    else mma_ss(dd, da + (uint64_t)(2 * (g & 3)), db + (uint64_t)((g & 3) * (b_mn ? 128 : 2)), idesc, acc);
                }
            }
            t1 = clock64();
            mma_commit(&bar);
        }
        __syncwarp();
        const bool ok = mbar_wait(&bar, 0, abort_flag, 400000000LL);
        const long long t2 = clock64();
        if (tid == 0) { out[0] = ok ? t2 - t0 : -1; out[1] = t1 - t0; }
        if (tid == 32) { out[2] = ok ? t2 - t0 : -1; out[3] = t1 - t0; }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}
}  // namespace hdt

// Diagnostics: see k_debug_mma_rate.  out2 (host): cycles until the last MMA completed, cycles of the issue loop.
extern "C" int hdt_debug_mma_rate(int32_t n, int32_t reps, int32_t per_group, int32_t mode, int32_t b_mn, int64_t *out2) {
    if (!out2 || n < 16 || n > 128 || n % 16 || reps < 1 || reps > 100000 || per_group < 1 || per_group > 64 || mode < 0 || mode > 7)
        return hdt::set_error(HDT_ERR_INVALID_ARG, "hdt_debug_mma_rate: bad arguments");
    long long *d = nullptr;
    HDT_CUDA_CHECK(cudaMalloc(&d, 32));
    const int smem = 4 * 16384;
    HDT_CUDA_CHECK(cudaFuncSetAttribute(hdt::k_debug_mma_rate, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    hdt::k_debug_mma_rate<<<1, 128, smem>>>(n, reps, per_group, mode, b_mn, d);
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(out2, d, 16, cudaMemcpyDeviceToHost);
    cudaFree(d);
    if (e != cudaSuccess) return hdt::set_error(HDT_ERR_CUDA, "hdt_debug_mma_rate: %s", cudaGetErrorString(e));
    return HDT_OK;
}

namespace hdt {
// Timing probe of TMEM loads: `warps` warps (lane quarter = warp % 4) each do `reps` rounds of `per_round`
// tcgen05.ld (32 lanes x 16 columns) followed by one tcgen05.wait::ld, while (mma != 0) warp 31 keeps the
// tensor pipe busy with N = 64 MMAs accumulating into other TMEM columns.  out[w] = cycles of warp w's loop.
__global__ void __launch_bounds__(1024) k_debug_tmem_ld(int warps, int reps, int per_round, int mma, long long *out) {
    extern __shared__ __align__(1024) uint8_t sm[];
    __shared__ uint64_t bar;
    __shared__ uint32_t slot;
    __shared__ int abort_s, stop_s;
    volatile int *abort_flag = &abort_s;
    volatile int *stop = &stop_s;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int i = tid; i < 4 * 16384 / 4; i += blockDim.x) ((uint32_t *)sm)[i] = 0x3c003c00u;
    if (tid == 0) { mbar_init(&bar, 1); *abort_flag = 0; *stop = 0; fence_mbar_init(); }
    fence_proxy_async_smem();
    if (warp == 0) tmem_alloc(&slot, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = slot;
    if (warp < warps && mma >= 2) {
        // mma = 2 + n: warp 31 issues n MMAs into columns 256..383 and commits; the loading warps wait for the
        // commit's barrier and then time `reps` rounds of loads FROM THOSE COLUMNS (out[w] = cycles of the rounds,
        // out[16 + w] = cycles the wait for the barrier took after the loop's start)
        const uint32_t base = tmem + 256u + ((uint32_t)((warp & 3) * 32) << 16) + 16u * ((warp >> 2) & 7);
        uint32_t acc = 0;
        const long long ta = clock64();
        (void)mbar_wait(&bar, 0, abort_flag, 400000000LL);
        tc_fence_after();
        const long long t0 = clock64();
        for (int r = 0; r < reps; ++r) {
            uint32_t v[4][16];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (k < per_round) tmem_ld16(base + 64u * (k & 1), v[k]);
            tmem_wait_ld();
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (k < per_round) acc ^= v[k][0] ^ v[k][15];
        }
        const long long t1 = clock64();
        if (lane == 0) { out[warp] = t1 - t0 + (acc == 0x12345678u ? 1 : 0); if (warp < 16) out[16 + warp] = t0 - ta; }
    } else if (warp == 31 && mma >= 2) {
        if (elect_one()) {
            const uint32_t idesc = idesc_bf16(64, false, true);
            const uint64_t da = smem_desc(smem_u32(sm), 0, 1024);
            const uint64_t db = smem_desc(smem_u32(sm) + 2 * 16384, 16384, 1024);
            for (int g = 0; g < mma - 2; ++g) mma_ss(tmem + 256u + 64u * (g & 1), da + (uint64_t)(2 * (g & 3)), db + (uint64_t)((g & 3) * 128), idesc, g > 1);
            mma_commit(&bar);
        }
        __syncwarp();
    } else if (warp < warps) {
        const uint32_t base = tmem + ((uint32_t)((warp & 3) * 32) << 16) + 16u * ((warp >> 2) & 7);
        uint32_t acc = 0;
        const long long t0 = clock64();
        for (int r = 0; r < reps; ++r) {
            uint32_t v[4][16];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (k < per_round) tmem_ld16(base + 128u * (k & 1), v[k]);
            tmem_wait_ld();
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (k < per_round) acc ^= v[k][0] ^ v[k][15];
        }
        const long long t1 = clock64();
        if (lane == 0) out[warp] = t1 - t0 + (acc == 0x12345678u ? 1 : 0);
        __syncwarp();
        if (warp == 0 && lane == 0) *stop = 1;
    } else if (warp == 31 && mma == 1) {
        if (elect_one()) {
            const uint32_t idesc = idesc_bf16(64, false, true);
            const uint64_t da = smem_desc(smem_u32(sm), 0, 1024);
            const uint64_t db = smem_desc(smem_u32(sm) + 2 * 16384, 16384, 1024);
            int n = 0;
            while (!*stop && n < 20000) {
                for (int g = 0; g < 8; ++g) mma_ss(tmem + 256u + 64u * (g & 1), da + (uint64_t)(2 * (g & 3)), db + (uint64_t)((g & 3) * 128), idesc, 1);
                n += 8;
            }
            mma_commit(&bar);
        }
        __syncwarp();
        (void)mbar_wait(&bar, 0, abort_flag, 400000000LL);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}
}  // namespace hdt

// Diagnostics: see k_debug_tmem_ld.  out32 (host): cycles of each loading warp's loop.
extern "C" int hdt_debug_tmem_ld(int32_t warps, int32_t reps, int32_t per_round, int32_t mma, int64_t *out32) {
    if (!out32 || warps < 1 || warps > 28 || reps < 1 || reps > 100000 || per_round < 1 || per_round > 4)
        return hdt::set_error(HDT_ERR_INVALID_ARG, "hdt_debug_tmem_ld: bad arguments");
    long long *d = nullptr;
    HDT_CUDA_CHECK(cudaMalloc(&d, 256));
    HDT_CUDA_CHECK(cudaMemset(d, 0, 256));
    const int smem = 4 * 16384;
    HDT_CUDA_CHECK(cudaFuncSetAttribute(hdt::k_debug_tmem_ld, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    hdt::k_debug_tmem_ld<<<1, 1024, smem>>>(warps, reps, per_round, mma, d);
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(out32, d, 256, cudaMemcpyDeviceToHost);
    cudaFree(d);
    if (e != cudaSuccess) return hdt::set_error(HDT_ERR_CUDA, "hdt_debug_tmem_ld: %s", cudaGetErrorString(e));
    return HDT_OK;
}
