// Stand-alone evaluators of the kernels' integer building blocks, for exhaustive checks on the device:
// the integer sigmoid / tanh over the whole int16 domain, and the integer layer norm of one row.
// They run the same device functions (qmath.cuh) that the recurrent kernel inlines.
#include <cuda_runtime.h>

#include "../../include/qlstm.h"
#include "../../include/qlstm_debug.h"
#include "qmath.cuh"

namespace ql {

__global__ void k_eval_activations(int m, int16_t *sig, int16_t *tnh)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 65536) return;
    const int32_t x = i - 32768;
    sig[i] = (int16_t)sigmoid_q_fast(x, m);
    tnh[i] = (int16_t)tanh_q_fast(x, m);
}

__global__ void k_eval_layernorm_row(const int16_t *q, int n, const int16_t *L, const int32_t *b, Scale eff, int16_t *out)
{
    __shared__ long long s_sum[32], s_sq[32];
    __shared__ LnRow row;
    long long sum = 0, sq = 0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) { long long v = q[i]; sum += v; sq += v * v; }
    for (int o = 16; o > 0; o >>= 1) { sum += __shfl_down_sync(0xffffffffu, sum, o); sq += __shfl_down_sync(0xffffffffu, sq, o); }
    if ((threadIdx.x & 31) == 0) { s_sum[threadIdx.x >> 5] = sum; s_sq[threadIdx.x >> 5] = sq; }
    __syncthreads();
    if (threadIdx.x == 0) {
        long long a = 0, c = 0;
        for (int w = 0; w < (int)(blockDim.x + 31) / 32; ++w) { a += s_sum[w]; c += s_sq[w]; }
        row = make_ln_row(ln_stats(a, c, n));
    }
    __syncthreads();
    const FastScale f = make_fast_scale(eff);
    for (int i = threadIdx.x; i < n; i += blockDim.x) out[i] = (int16_t)ln_apply_fast(q[i], row, L[i], b[i], eff, f);
}

}  // namespace ql

extern "C" {

int qlstm_eval_activations(int cell_int_bits, int16_t *sigmoid_dev, int16_t *tanh_dev, void *cuda_stream)
{
    if (cell_int_bits < 0 || cell_int_bits > 15 || !sigmoid_dev || !tanh_dev) return QLSTM_ERR_ARG;
    ql::k_eval_activations<<<256, 256, 0, (cudaStream_t)cuda_stream>>>(cell_int_bits, sigmoid_dev, tanh_dev);
    return cudaGetLastError() == cudaSuccess ? QLSTM_OK : QLSTM_ERR_CUDA;
}

int qlstm_eval_layernorm_row(const int16_t *q_dev, int n, const int16_t *L_dev, const int32_t *b_dev, qlstm_scale_t eff_ln,
                             int16_t *out_dev, void *cuda_stream)
{
    if (!q_dev || !L_dev || !b_dev || !out_dev || n <= 0 || n > 8191) return QLSTM_ERR_ARG;
    if (eff_ln.multiplier != 0 && (eff_ln.multiplier < (1 << 30) || eff_ln.shift < -31 || eff_ln.shift > 30)) return QLSTM_ERR_ARG;
    ql::k_eval_layernorm_row<<<1, 256, 0, (cudaStream_t)cuda_stream>>>(q_dev, n, L_dev, b_dev,
                                                                       ql::Scale{eff_ln.multiplier, eff_ln.shift}, out_dev);
    return cudaGetLastError() == cudaSuccess ? QLSTM_OK : QLSTM_ERR_CUDA;
}

}  // extern "C"
