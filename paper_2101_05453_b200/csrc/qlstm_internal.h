// Internal types shared by the host API and the kernels of libqlstm.so.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "qmath.cuh"

namespace ql {

enum { F_PROJECTION = 1, F_PEEPHOLE = 2, F_LAYERNORM = 4, F_CIFG = 8 };

// Device view of one layer.  Gate rows are interleaved per cell: row n = u * G + gi, where gi
// runs over the active gates (i, f, z, o; with CIFG only f, z, o) and gate_id[gi] is the
// canonical gate number (0 i, 1 f, 2 z, 3 o).  One CTA that owns a range of cells therefore
// owns a contiguous range of rows of W, R and of every per-row vector.
struct LayerParams {
    int I, C, O, G, N;                 // N = C * G
    uint32_t flags;
    int m_bits;                        // cell format Q_{m.15-m}
    int zp_m, zp_h;
    int gate_id[4];
    int slot_of_gate[4];               // canonical gate -> gi, or -1
    const int8_t *W;                   // [N][I]
    const int8_t *R;                   // [N][O]
    const int8_t *Wproj;               // [O][C]
    const int32_t *bx;                 // [N]  -zp_x * sum_j W[n][j]
    const int32_t *bh;                 // [N]  (bias without LN) - zp_h * sum_k R[n][k]
    const int32_t *bp;                 // [O]  b_proj - zp_m * sum_u Wproj[p][u]
    const int16_t *P;                  // [N]  peephole weights, 0 where the gate has none
    const int16_t *L;                  // [N]  layer-norm weights
    const int32_t *bln;                // [N]  layer-norm bias
    Scale eff_x[4], eff_h[4], eff_c[4], eff_ln[4];   // indexed by gi
    Scale eff_m, eff_proj;
};

// Views into one trace record (see include/qlstm.h); all null when tracing is off.
struct TraceRec {
    int32_t *acc, *pacc;
    int16_t *xg, *pre, *ain, *gate, *c;
    int8_t *m, *h;
};

inline size_t trace_record_bytes(int B, int C, int O)
{
    size_t bc = (size_t)B * C, bo = (size_t)B * O;
    size_t n = 16 * bc + 4 * bo + 4 * (8 * bc) + 2 * bc + bc + bo;
    return (n + 15) & ~(size_t)15;
}

inline TraceRec trace_view(uint8_t *p, int B, int C, int O)
{
    size_t bc = (size_t)B * C, bo = (size_t)B * O;
    TraceRec v;
    v.acc = (int32_t *)p;   p += 16 * bc;
    v.pacc = (int32_t *)p;  p += 4 * bo;
    v.xg = (int16_t *)p;    p += 8 * bc;
    v.pre = (int16_t *)p;   p += 8 * bc;
    v.ain = (int16_t *)p;   p += 8 * bc;
    v.gate = (int16_t *)p;  p += 8 * bc;
    v.c = (int16_t *)p;     p += 2 * bc;
    v.m = (int8_t *)p;      p += bc;
    v.h = (int8_t *)p;
    return v;
}

// Scratch of the simple (one launch per phase) recurrent path.
struct SimpleScratch {
    int16_t *pre;       // [B][N] gate sums
    int32_t *po;        // [B][C] X_o + H_o before the peephole term on c^t
    int64_t *stats;     // [B][G][2] layer-norm mean, sigma
    int8_t *m;          // [B][C]
};

// ---- launchers implemented in simple_kernels.cu --------------------------------------------
cudaError_t launch_projection_simple(const LayerParams &p, const int8_t *x, int rows, int16_t *X,
                                     cudaStream_t st);
// runs T steps; returns the number of kernel launches through *launches
cudaError_t launch_recurrent_simple(const LayerParams &p, const int16_t *X, int T, int B, int8_t *h,
                                    int16_t *c, int8_t *y, const SimpleScratch &s, uint8_t *trace,
                                    size_t trace_stride, cudaStream_t st, int *launches);

}  // namespace ql
