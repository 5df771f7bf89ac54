// Stand-alone evaluators of the kernels' integer building blocks, for exhaustive checks on the device:
// the integer sigmoid / tanh over the whole int16 domain, and the integer layer norm of one row.
// They run the same device functions (qmath.cuh) that the recurrent kernel inlines.
#include <cuda_runtime.h>

#include "../../include/qlstm.h"
#include "../../include/qlstm_debug.h"
#include "act_table.cuh"
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

// The memoised nonlinearities through the lookup code of the recurrent kernel: the blob is copied into shared memory
// as that kernel's bulk copy does, then every int16 input is looked up.
__global__ void k_eval_activation_tables(const uint8_t *blob, ActTabLayout lay, int16_t *sig, int16_t *tz, int16_t *tc)
{
    extern __shared__ __align__(16) uint8_t tab_s[];
    for (uint32_t i = threadIdx.x; i < lay.bytes / 16; i += blockDim.x)
        reinterpret_cast<uint4 *>(tab_s)[i] = reinterpret_cast<const uint4 *>(blob)[i];
    __syncthreads();
    const ActTabs at = make_act_tabs((uint32_t)__cvta_generic_to_shared(tab_s), lay);
    for (int i = threadIdx.x; i < 65536; i += blockDim.x) {
        const int32_t x = i - 32768;
        sig[i] = (int16_t)tab_sigmoid(at, x);
        tz[i] = (int16_t)tab_tanh_gate(at, x);
        tc[i] = (int16_t)tab_tanh_cell(at, x);
    }
}

}  // namespace ql

extern "C" {

int qlstm_eval_activation_tables(int cell_int_bits, int max_bytes, int16_t *sigmoid_dev, int16_t *tanh_gate_dev,
                                 int16_t *tanh_cell_dev, int *layout_out7, void *cuda_stream)
{
    if (cell_int_bits < 0 || cell_int_bits > 15 || max_bytes < 0 || max_bytes > 128 * 1024 || !sigmoid_dev || !tanh_gate_dev ||
        !tanh_cell_dev || !layout_out7)
        return QLSTM_ERR_ARG;
    int *layout_out6 = layout_out7;
    uint8_t *blob = nullptr;
    ql::ActTabLayout lay;
    if (!ql::act_tables_build(cell_int_bits, (size_t)max_bytes, &blob, &lay)) return QLSTM_ERR_CUDA;
    layout_out6[0] = (int)lay.bytes; layout_out6[1] = (int)lay.tz_off; layout_out6[2] = (int)lay.tc_off;
    layout_out6[3] = lay.tz_amax; layout_out6[4] = lay.tc_amax; layout_out6[5] = lay.tc_mode; layout_out7[6] = lay.sig_packed;
    if (!blob) return QLSTM_OK;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int rc = QLSTM_OK;
    if (cudaFuncSetAttribute(ql::k_eval_activation_tables, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lay.bytes) != cudaSuccess)
        rc = QLSTM_ERR_CUDA;
    if (rc == QLSTM_OK) {
        ql::k_eval_activation_tables<<<1, 1024, lay.bytes, st>>>(blob, lay, sigmoid_dev, tanh_gate_dev, tanh_cell_dev);
        if (cudaGetLastError() != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) rc = QLSTM_ERR_CUDA;
    }
    cudaFree(blob);
    return rc;
}

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
