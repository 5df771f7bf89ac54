// Integer layer norm over many rows with no allocation at all.
//
// Some callers of this library may not allocate device memory when they need a result: a per-frame
// audio loop that must not take the runtime's allocator lock (cudaMalloc and cudaFree serialise against
// the whole device and can wait behind unrelated work), a process that has already given every byte of
// the GPU to its own arena, or a plug-in whose host forbids allocation inside its processing callback.
// For them this entry point keeps the only intermediate it needs - the per-row statistics that sit
// between the reduction pass and the normalisation pass - in a fixed array that is part of the library
// image.  Every device that loads the library holds that array (64 KiB) until the process exits.
#include <cuda_runtime.h>

#include "../../include/qlstm.h"
#include "qmath.cuh"

namespace {

constexpr int MAX_ROWS = 4096;            // rows per call; 4096 rows x 4 gate slots would be one step at batch 1024

// [row][0] = mean, [row][1] = sigma of Section 3.2.6.  File-scope device storage: in host code this name
// is only a handle for cudaGetSymbolAddress, never an address a kernel could use.
static __device__ __align__(256) long long g_row_stats[MAX_ROWS][2];

constexpr int MAX_DEVICES = 64;
long long (*g_stats_ptr[MAX_DEVICES])[2] = {};   // device address of g_row_stats, per device, set on first use

// pass 1: one block per row -> statistics into the static array (every entry used by pass 2 is overwritten
// here first, so nothing left by an earlier call is ever read)
__global__ void k_rows_stats(const int16_t *q, int n, long long (*stats)[2])
{
    __shared__ long long s_sum[8], s_sq[8];
    const int16_t *row = q + (size_t)blockIdx.x * n;
    long long sum = 0, sq = 0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) { long long v = row[i]; sum += v; sq += v * v; }
    for (int o = 16; o > 0; o >>= 1) { sum += __shfl_down_sync(0xffffffffu, sum, o); sq += __shfl_down_sync(0xffffffffu, sq, o); }
    if ((threadIdx.x & 31) == 0) { s_sum[threadIdx.x >> 5] = sum; s_sq[threadIdx.x >> 5] = sq; }
    __syncthreads();
    if (threadIdx.x == 0) {
        long long a = 0, c = 0;
        for (int w = 0; w < (int)blockDim.x / 32; ++w) { a += s_sum[w]; c += s_sq[w]; }
        ql::LnStats st = ql::ln_stats(a, c, n);
        stats[blockIdx.x][0] = st.mean;
        stats[blockIdx.x][1] = st.sigma;
    }
}

// pass 2: one thread per element
__global__ void k_rows_apply(const int16_t *q, int rows, int n, const int16_t *L, const int32_t *b, ql::Scale eff,
                             const long long (*stats)[2], int16_t *out)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)rows * n) return;
    const int r = (int)(idx / n), i = (int)(idx % n);
    ql::LnStats st{stats[r][0], stats[r][1]};
    out[idx] = (int16_t)ql::ln_apply_fast(q[idx], ql::make_ln_row(st), L[i], b[i], eff, ql::make_fast_scale(eff));
}

}  // namespace

extern "C" int qlstm_layernorm_rows_static(const int16_t *q_dev, int rows, int n, const int16_t *L_dev,
                                           const int32_t *b_dev, qlstm_scale_t eff_ln, int16_t *out_dev,
                                           void *cuda_stream)
{
    if (rows < 0 || n <= 0 || n > 8191) return QLSTM_ERR_ARG;
    // same window as qlstm_create: multiplier 0 or in [2^30, 2^31), shift in [-31, 30] (beyond it the shifts are undefined)
    if (eff_ln.multiplier != 0 && (eff_ln.multiplier < (1 << 30) || eff_ln.shift < -31 || eff_ln.shift > 30)) return QLSTM_ERR_ARG;
    if (rows > MAX_ROWS) return QLSTM_ERR_DIM;                       // beyond the fixed scratch
    if (rows == 0) return QLSTM_OK;
    if (!q_dev || !L_dev || !b_dev || !out_dev) return QLSTM_ERR_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return QLSTM_ERR_CUDA;
    if (!g_stats_ptr[dev]) {
        // set-up, once per device, with that device current: resolve the array's device address
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_row_stats) != cudaSuccess || !p) return QLSTM_ERR_CUDA;
        g_stats_ptr[dev] = (long long (*)[2])p;
    }
    long long (*stats)[2] = g_stats_ptr[dev];
    cudaStream_t st = (cudaStream_t)cuda_stream;
    k_rows_stats<<<rows, 256, 0, st>>>(q_dev, n, stats);
    const size_t total = (size_t)rows * n;
    k_rows_apply<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(q_dev, rows, n, L_dev, b_dev,
                                                                  ql::Scale{eff_ln.multiplier, eff_ln.shift}, stats, out_dev);
    return cudaGetLastError() == cudaSuccess ? QLSTM_OK : QLSTM_ERR_CUDA;
}
