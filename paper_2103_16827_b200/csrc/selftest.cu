// Self-test of the bounded device-side wait: one small CTA goes through the set-up and teardown the
// tensor-core kernels share (mbarrier init, TMEM allocation, abort flag, TMEM release) and waits on an
// mbarrier that nothing ever arrives on.  The wait gives up after the requested time, raises the
// sticky status word and the CTA leaves through the normal teardown, so the context stays usable.
// The wait ends by construction; no pipeline is starved and nothing can hang.
#include <cstdio>

#include "qasr_host.h"
#include "sm100_ptx.cuh"

namespace qasr {
namespace selftest {

constexpr int TMEM_COLS = 32;

__global__ void __launch_bounds__(64, 1)
wait_timeout_kernel(unsigned* status, unsigned long long limit_ns) {
    __shared__ uint64_t never_arrives;
    __shared__ uint32_t tmem_base_slot;
    __shared__ volatile int abort_flag;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&never_arrives), 1);
        abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_base_slot), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    if (warp == 0) {
        // the whole warp polls, as the MMA warps of the real kernels do
        bool ok = ptx::mbar_wait(ptx::smem_u32(&never_arrives), 0, &abort_flag, status, limit_ns);
        ok = __all_sync(0xffffffffu, ok);
        (void)ok;
    }
    // teardown, as in the real kernels
    ptx::tc_fence_before();
    __syncthreads();
    if (abort_flag) {
        if (threadIdx.x == 0)
            for (int i = 0; i < 4; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ---------------------------------------------------------------------------------------------
// Measured int8 tensor-core peak: every SM issues back-to-back tcgen05.mma kind::i8 instructions
// (M = 128, N = 256, K = 32) on operands that stay fixed in shared memory; no loads in the loop.
// ---------------------------------------------------------------------------------------------
constexpr int PEAK_N = 256;
constexpr int PEAK_A_BYTES = 128 * 128;       // 128 rows x 128 bytes of K, 128-byte swizzle
constexpr int PEAK_B_BYTES = PEAK_N * 128;

__global__ void __launch_bounds__(128, 1)
int8_peak_kernel(int kblocks, unsigned* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t done;
    __shared__ uint32_t tmem_base_slot;
    __shared__ volatile int abort_flag;
    const int warp = threadIdx.x >> 5;
    // operand bytes: any values do (the products are never read), but not all equal, so that the
    // multipliers see changing data as they do in the real kernels
    for (int i = threadIdx.x; i < (PEAK_A_BYTES + PEAK_B_BYTES) / 4; i += blockDim.x)
        reinterpret_cast<uint32_t*>(smem)[i] = (uint32_t)i * 2654435761u + blockIdx.x;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&done), 1);
        abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&tmem_base_slot), 512);
        ptx::tmem_relinquish();
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    if (warp == 0) {
        const uint32_t idesc = ptx::idesc_i8(128, PEAK_N, 0, 0);
        const uint64_t a_desc = ptx::smem_desc(ptx::smem_u32(smem), 16, 1024, ptx::SWIZZLE_128B);
        const uint64_t b_desc = ptx::smem_desc(ptx::smem_u32(smem + PEAK_A_BYTES), 16, 1024, ptx::SWIZZLE_128B);
        if (ptx::elect_one()) {
            for (int kb = 0; kb < kblocks; ++kb) {
                const uint32_t d = tmem_base + (kb & 1) * 256;     // two accumulators, alternating
#pragma unroll
                for (int j = 0; j < 4; ++j) ptx::mma_i8(d, a_desc + 2 * j, b_desc + 2 * j, idesc, 1u);
            }
            ptx::tc_commit(ptx::smem_u32(&done));
        }
        __syncwarp();
        bool ok = ptx::mbar_wait(ptx::smem_u32(&done), 0, &abort_flag, status);
        ok = __all_sync(0xffffffffu, ok);
        (void)ok;
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace selftest
}  // namespace qasr

extern "C" int qasr_measure_int8_tensor_peak(qasr_ctx* ctx, int kblocks, float* ms, double* ops) {
    if (!ctx || !ms || !ops) return QASR_ERR_NULL;
    if (kblocks < 1 || kblocks > (1 << 20)) {
        snprintf(ctx->err, sizeof(ctx->err), "qasr_measure_int8_tensor_peak: kblocks=%d must be in [1, 2^20]", kblocks);
        return QASR_ERR_SHAPE;
    }
    if (ctx->cc_major != 10) {
        snprintf(ctx->err, sizeof(ctx->err), "qasr_measure_int8_tensor_peak needs an sm_100 device");
        return QASR_ERR_CUDA;
    }
    using namespace qasr::selftest;
    const size_t smem = 1024 + PEAK_A_BYTES + PEAK_B_BYTES;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = cudaSetDevice(ctx->device);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(int8_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    if (e == cudaSuccess) {
        int8_peak_kernel<<<ctx->sm_count, 128, smem, ctx->stream>>>(8, ctx->d_status);      // warm-up
        cudaEventRecord(e0, ctx->stream);
        int8_peak_kernel<<<ctx->sm_count, 128, smem, ctx->stream>>>(kblocks, ctx->d_status);
        cudaEventRecord(e1, ctx->stream);
        ctx->launches += 2;
        e = cudaGetLastError();
        if (e == cudaSuccess) e = cudaEventSynchronize(e1);
        if (e == cudaSuccess) e = cudaEventElapsedTime(ms, e0, e1);
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (e != cudaSuccess) {
        snprintf(ctx->err, sizeof(ctx->err), "qasr_measure_int8_tensor_peak: %s", cudaGetErrorString(e));
        return QASR_ERR_CUDA;
    }
    *ops = 2.0 * 128.0 * PEAK_N * 128.0 * (double)kblocks * (double)ctx->sm_count;
    return QASR_OK;
}

extern "C" int qasr_selftest_wait_timeout(qasr_ctx* ctx, unsigned limit_us) {
    if (!ctx) return QASR_ERR_NULL;
    if (limit_us < 1 || limit_us > 1000000u) {
        snprintf(ctx->err, sizeof(ctx->err), "qasr_selftest_wait_timeout: limit_us=%u must be in [1, 1000000]", limit_us);
        return QASR_ERR_SHAPE;
    }
    if (ctx->cc_major != 10) {
        snprintf(ctx->err, sizeof(ctx->err), "qasr_selftest_wait_timeout needs an sm_100 device");
        return QASR_ERR_CUDA;
    }
    if (cudaSetDevice(ctx->device) != cudaSuccess) {
        cudaGetLastError();
        return QASR_ERR_CUDA;
    }
    ctx->launches++;
    qasr::selftest::wait_timeout_kernel<<<1, 64, 0, ctx->stream>>>(ctx->d_status, (unsigned long long)limit_us * 1000ull);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        snprintf(ctx->err, sizeof(ctx->err), "wait_timeout_kernel launch failed: %s", cudaGetErrorString(e));
        return QASR_ERR_CUDA;
    }
    return QASR_OK;
}
