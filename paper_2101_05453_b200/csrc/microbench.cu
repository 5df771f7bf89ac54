// Two measurements the roofline statements rest on, as kernels of their own (neither is on the product path):
//
//   qlstm_debug_mma_i8_peak     back-to-back tcgen05.mma kind::i8 (M128 N256 K32) from operands resident in shared
//                               memory into two tensor-memory accumulators, on every SM at once: the issue-rate peak of
//                               the int8 tensor path as this library drives it.  There is no measured int8 figure for
//                               the device otherwise (only bf16), so this is the denominator "what the MMA pipe can do".
//   qlstm_debug_barrier_latency the grid-wide barrier of the persistent recurrent kernel (release-add on one counter,
//                               acquire polling by one thread per block) executed n times in a row with nothing in
//                               between: the floor that every phase boundary of a time step pays.
//
// Both waits are bounded; on expiry the kernel stores an error flag and returns.
#include <cuda_runtime.h>

#include "../../include/qlstm.h"
#include "../../include/qlstm_debug.h"
#include "sm100_ptx.cuh"

namespace ql {

namespace {

constexpr int MB_THREADS = 128;
constexpr int MB_N = 256;
constexpr int MB_A_BYTES = 128 * 128, MB_B_BYTES = MB_N * 128;      // one 128-byte k-block of each operand

__global__ void __launch_bounds__(MB_THREADS, 1) k_mma_i8_peak(int iters, int *err)
{
    extern __shared__ uint8_t mb_smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)mb_smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t done;
    __shared__ uint32_t tmem_base_s;
    uint8_t *A_s = smem, *B_s = smem + MB_A_BYTES;
    for (int i = threadIdx.x; i < (MB_A_BYTES + MB_B_BYTES) / 16; i += MB_THREADS)
        reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0x01010101u, 0x01010101u, 0x01010101u, 0x01010101u);
    if (threadIdx.x == 0) {
        ptx::mbar_init(&done, 1);
        ptx::fence_barrier_init();
    }
    if (threadIdx.x < 32) {
        ptx::tmem_alloc(&tmem_base_s, 512);
        ptx::tmem_relinquish();
    }
    ptx::fence_proxy_async();                 // the operands were written by ordinary stores; the MMA reads them as async proxy
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    if (threadIdx.x == 0) {
        const uint32_t idesc = ptx::idesc_i8(128, MB_N);
        const uint64_t a_desc = ptx::smem_desc_k_sw128(ptx::smem_u32(A_s));
        const uint64_t b_desc = ptx::smem_desc_k_sw128(ptx::smem_u32(B_s));
        for (int it = 0; it < iters; ++it) {
            const uint32_t d = tmem_base + (uint32_t)((it & 1) * MB_N);
#pragma unroll
            for (int k = 0; k < 4; ++k) ptx::mma_i8_ss(d, a_desc + 2 * k, b_desc + 2 * k, idesc, it >= 2 || k != 0);
        }
        ptx::mma_commit(&done);
        bool ok = false;
        for (uint32_t i = 0; i < 200000u && !ok; ++i) ok = ptx::mbar_try_wait_parked(&done, 0, 20000u);    // <= 4 s
        if (!ok) atomicExch(err, 1);
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, 512);
    }
}

__global__ void __launch_bounds__(128, 1) k_barrier_latency(unsigned *bar, int n, unsigned long long limit_ns, int *err)
{
    __shared__ int abort_s;
    if (threadIdx.x == 0) abort_s = 0;
    __syncthreads();
    for (int e = 1; e <= n; ++e) {
        __syncthreads();
        if (threadIdx.x == 0) {
            const unsigned target = (unsigned)e * gridDim.x;
            asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(bar) : "memory");
            unsigned long long t0;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0)::"memory");
            unsigned v, spins = 0;
            for (;;) {
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(bar) : "memory");
                if (v >= target) break;
                if ((++spins & 63u) == 0u) {
                    unsigned a;
                    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(a) : "l"(bar + 1) : "memory");
                    unsigned long long now;
                    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(now)::"memory");
                    if (a != 0u || now - t0 > limit_ns) { atomicExch(bar + 1, 1u); abort_s = 1; break; }
                }
            }
        }
        __syncthreads();
        if (abort_s) break;
    }
    if (abort_s && threadIdx.x == 0) atomicExch(err, 1);
}

}  // namespace
}  // namespace ql

extern "C" {

int qlstm_debug_mma_i8_peak(int device, int iters, double *tops_out)
{
    if (!tops_out || iters < 16 || iters > (1 << 22)) return QLSTM_ERR_ARG;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess || prop.major != 10) return QLSTM_ERR_CUDA;
    if (cudaSetDevice(device) != cudaSuccess) return QLSTM_ERR_CUDA;
    const size_t smem = 1024 + ql::MB_A_BYTES + ql::MB_B_BYTES;
    if (cudaFuncSetAttribute(ql::k_mma_i8_peak, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return QLSTM_ERR_CUDA;
    int *err = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    if (cudaMalloc(&err, sizeof(int)) != cudaSuccess) return QLSTM_ERR_NOMEM;
    cudaMemset(err, 0, sizeof(int));
    cudaEventCreate(&a);
    cudaEventCreate(&b);
    const int grid = prop.multiProcessorCount;
    float best = 0.f;
    int rc = QLSTM_OK;
    for (int rep = 0; rep < 4 && rc == QLSTM_OK; ++rep) {                        // first repetition is the warm-up
        cudaEventRecord(a, 0);
        ql::k_mma_i8_peak<<<grid, ql::MB_THREADS, smem, 0>>>(iters, err);
        cudaEventRecord(b, 0);
        if (cudaEventSynchronize(b) != cudaSuccess || cudaGetLastError() != cudaSuccess) { rc = QLSTM_ERR_CUDA; break; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, a, b);
        if (rep > 0 && (best == 0.f || ms < best)) best = ms;
    }
    int herr = 0;
    if (rc == QLSTM_OK && cudaMemcpy(&herr, err, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) rc = QLSTM_ERR_CUDA;
    if (rc == QLSTM_OK && herr) rc = QLSTM_ERR_TIMEOUT;
    if (rc == QLSTM_OK) *tops_out = (double)grid * iters * 4.0 * 2.0 * 128.0 * ql::MB_N * 32.0 / (best * 1e-3) / 1e12;
    cudaEventDestroy(a);
    cudaEventDestroy(b);
    cudaFree(err);
    return rc;
}

int qlstm_debug_barrier_latency(int device, int n_barriers, double *us_per_barrier_out)
{
    if (!us_per_barrier_out || n_barriers < 1 || n_barriers > 1000000) return QLSTM_ERR_ARG;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return QLSTM_ERR_CUDA;
    if (cudaSetDevice(device) != cudaSuccess) return QLSTM_ERR_CUDA;
    unsigned *bar = nullptr;
    int *err = nullptr;
    if (cudaMalloc(&bar, 64) != cudaSuccess) return QLSTM_ERR_NOMEM;
    if (cudaMalloc(&err, sizeof(int)) != cudaSuccess) { cudaFree(bar); return QLSTM_ERR_NOMEM; }
    cudaMemset(err, 0, sizeof(int));
    cudaEvent_t a = nullptr, b = nullptr;
    cudaEventCreate(&a);
    cudaEventCreate(&b);
    const int grid = prop.multiProcessorCount;
    unsigned long long limit = 1000000000ull;
    void *args[] = {(void *)&bar, (void *)&n_barriers, (void *)&limit, (void *)&err};
    float best = 0.f;
    int rc = QLSTM_OK;
    for (int rep = 0; rep < 4 && rc == QLSTM_OK; ++rep) {
        cudaMemsetAsync(bar, 0, 64, 0);
        cudaEventRecord(a, 0);
        cudaError_t e = cudaLaunchCooperativeKernel((const void *)ql::k_barrier_latency, dim3(grid), dim3(128), args, 0, 0);
        cudaEventRecord(b, 0);
        if (e != cudaSuccess || cudaEventSynchronize(b) != cudaSuccess) { cudaGetLastError(); rc = QLSTM_ERR_CUDA; break; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, a, b);
        if (rep > 0 && (best == 0.f || ms < best)) best = ms;
    }
    int herr = 0;
    if (rc == QLSTM_OK && cudaMemcpy(&herr, err, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) rc = QLSTM_ERR_CUDA;
    if (rc == QLSTM_OK && herr) rc = QLSTM_ERR_TIMEOUT;
    if (rc == QLSTM_OK) *us_per_barrier_out = 1e3 * best / n_barriers;
    cudaEventDestroy(a);
    cudaEventDestroy(b);
    cudaFree(bar);
    cudaFree(err);
    return rc;
}

}  // extern "C"
