// Bidirectional integer LSTM (Section 7: uni- and bidirectional LSTMs are loops over the same cell).
//
// Two stacks read the same input sequence, one from t = 0 upwards and one from t = T - 1 downwards; the output at
// step t is the forward stack's h^t followed by the backward stack's h^t (the state it has after seeing x_{T-1}..x_t).
// Each direction is an ordinary stack handle; this file adds the two small kernels around them - the time reversal of
// the input and the interleaving of the two output sequences - and the workspaces they need.
#include <cuda_runtime.h>

#include <new>

#include "../../include/qlstm.h"

struct qlstm_bidir {
    qlstm_t *fwd = nullptr, *bwd = nullptr;
    int device = 0, max_T = 0, max_B = 0;
    int n_input = 0, o_fwd = 0, o_bwd = 0;
    int8_t *x_rev = nullptr;       // [max_T][max_B][n_input]
    int8_t *y_fwd = nullptr;       // [max_T][max_B][o_fwd]
    int8_t *y_bwd = nullptr;       // [max_T][max_B][o_bwd], in the backward stack's own time order
};

namespace {

// dst[t] = src[T - 1 - t] for row blocks of `row_bytes` bytes (a multiple of 16)
__global__ void k_reverse_time(const uint4 *__restrict__ src, uint4 *__restrict__ dst, int T, size_t chunks_per_step)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)T * chunks_per_step) return;
    const size_t t = i / chunks_per_step, c = i - t * chunks_per_step;
    dst[i] = src[(size_t)(T - 1 - t) * chunks_per_step + c];
}

// y[t][b] = [ y_fwd[t][b] | y_bwd[T - 1 - t][b] ]
__global__ void k_concat_directions(const int8_t *__restrict__ yf, const int8_t *__restrict__ yb, int8_t *__restrict__ y, int T,
                                    int B, int of, int ob)
{
    const int o = of + ob;
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)T * B * o) return;
    const size_t row = i / o;
    const int col = (int)(i - row * o);
    const size_t t = row / B, b = row - t * B;
    y[i] = col < of ? yf[row * of + col] : yb[((size_t)(T - 1 - t) * B + b) * ob + (col - of)];
}

}  // namespace

extern "C" {

int qlstm_bidir_create(const qlstm_layer_t *fwd_layers, const qlstm_layer_t *bwd_layers, int n_layers, int max_T, int max_B,
                       int device, qlstm_bidir_t **out)
{
    if (!out) return QLSTM_ERR_ARG;
    *out = nullptr;
    if (!fwd_layers || !bwd_layers || n_layers <= 0 || max_T <= 0 || max_B <= 0) return QLSTM_ERR_ARG;
    if (fwd_layers[0].n_input != bwd_layers[0].n_input || fwd_layers[0].zp_x != bwd_layers[0].zp_x) return QLSTM_ERR_ARG;
    if (fwd_layers[0].n_input % 16 != 0) return QLSTM_ERR_DIM;                   // the reversal moves 16-byte chunks
    qlstm_bidir *q = new (std::nothrow) qlstm_bidir();
    if (!q) return QLSTM_ERR_NOMEM;
    q->device = device; q->max_T = max_T; q->max_B = max_B;
    q->n_input = fwd_layers[0].n_input;
    q->o_fwd = fwd_layers[n_layers - 1].n_output;
    q->o_bwd = bwd_layers[n_layers - 1].n_output;
    int rc = qlstm_create(fwd_layers, n_layers, max_T, max_B, device, &q->fwd);
    if (rc == QLSTM_OK) rc = qlstm_create(bwd_layers, n_layers, max_T, max_B, device, &q->bwd);
    if (rc == QLSTM_OK) {
        const size_t rows = (size_t)max_T * max_B;
        if (cudaMalloc(&q->x_rev, rows * q->n_input) != cudaSuccess || cudaMalloc(&q->y_fwd, rows * q->o_fwd) != cudaSuccess ||
            cudaMalloc(&q->y_bwd, rows * q->o_bwd) != cudaSuccess)
            rc = QLSTM_ERR_NOMEM;
    }
    if (rc != QLSTM_OK) { qlstm_bidir_destroy(q); return rc; }
    *out = q;
    return QLSTM_OK;
}

int qlstm_bidir_run(qlstm_bidir_t *q, const int8_t *x_dev, int T, int B, int8_t *h_fwd_dev, int16_t *c_fwd_dev, int8_t *h_bwd_dev,
                    int16_t *c_bwd_dev, int8_t *y_dev, void *cuda_stream)
{
    if (!q) return QLSTM_ERR_ARG;
    if (T < 0 || B < 0 || T > q->max_T || B > q->max_B) return QLSTM_ERR_ARG;
    if (T == 0 || B == 0) return QLSTM_OK;
    if (!x_dev || !h_fwd_dev || !c_fwd_dev || !h_bwd_dev || !c_bwd_dev || !y_dev) return QLSTM_ERR_ARG;
    if (((uintptr_t)x_dev & 15) != 0) return QLSTM_ERR_ARG;
    if (cudaSetDevice(q->device) != cudaSuccess) return QLSTM_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t chunks = (size_t)B * q->n_input / 16;
    const size_t total = (size_t)T * chunks;
    k_reverse_time<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(reinterpret_cast<const uint4 *>(x_dev),
                                                                    reinterpret_cast<uint4 *>(q->x_rev), T, chunks);
    if (cudaGetLastError() != cudaSuccess) return QLSTM_ERR_CUDA;
    int rc = qlstm_run(q->fwd, x_dev, T, B, h_fwd_dev, c_fwd_dev, q->y_fwd, nullptr, st);
    if (rc != QLSTM_OK) return rc;
    rc = qlstm_run(q->bwd, q->x_rev, T, B, h_bwd_dev, c_bwd_dev, q->y_bwd, nullptr, st);
    if (rc != QLSTM_OK) return rc;
    const size_t outs = (size_t)T * B * (q->o_fwd + q->o_bwd);
    k_concat_directions<<<(unsigned)((outs + 255) / 256), 256, 0, st>>>(q->y_fwd, q->y_bwd, y_dev, T, B, q->o_fwd, q->o_bwd);
    return cudaGetLastError() == cudaSuccess ? QLSTM_OK : QLSTM_ERR_CUDA;
}

int qlstm_bidir_last_status(qlstm_bidir_t *q)
{
    if (!q) return QLSTM_ERR_ARG;
    const int a = qlstm_last_status(q->fwd), b = qlstm_last_status(q->bwd);
    return a != QLSTM_OK ? a : b;
}

void qlstm_bidir_destroy(qlstm_bidir_t *q)
{
    if (!q) return;
    cudaSetDevice(q->device);
    cudaDeviceSynchronize();
    qlstm_destroy(q->fwd);
    qlstm_destroy(q->bwd);
    cudaFree(q->x_rev); cudaFree(q->y_fwd); cudaFree(q->y_bwd);
    delete q;
}

}  // extern "C"
