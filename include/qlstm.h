/*
 * qlstm — integer-only quantized LSTM forward pass on NVIDIA B200 (sm_100a).
 *
 * C ABI of libqlstm.so.  The library runs the integer execution graph of
 * "On the quantization of recurrent neural networks" (Li & Alvarez, arXiv 2101.05453):
 * int8 weights and activations, int32 accumulators, fixed-point (multiplier, shift)
 * rescaling, integer sigmoid / tanh, int16 cell state, and the projection, peephole,
 * layer-norm and CIFG variants (Section 2, Eq. 1-7; Section 3.2; Table 2).
 *
 * Conventions
 *   - affine quantization: real = scale * (q - zero_point); a requantize step adds the
 *     zero point of its output (Section 3.2.4, Section 6);
 *   - every rounding is to nearest, ties away from zero;
 *   - gate order i, f, z, o; matrices row-major [output unit][input unit];
 *   - "HOST" / "DEVICE" below says where a pointer must point.  Device pointers belong to
 *     the device given to qlstm_create.
 *   - every call returns 0 (QLSTM_OK) or a negative qlstm_error; nothing throws, aborts or prints.
 *     There is no CPU fallback: without a usable CUDA device every call fails with QLSTM_ERR_CUDA.
 */
#ifndef QLSTM_H
#define QLSTM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct qlstm qlstm_t;   /* opaque; owns the device copies of the weights and all workspaces */

/* Effective scale of a "rescale" node (Section 3.2.4: s_eff = 2^12 s_W s_x and the like):
 * real value = multiplier * 2^(shift - 31), multiplier in [2^30, 2^31) or 0.
 * rescale(x) = rounding_shift_right( sat_round_doubling_high_mul( sat32(x * 2^max(shift,0)), multiplier ), max(-shift,0) ). */
typedef struct { int32_t multiplier; int32_t shift; } qlstm_scale_t;

enum { QLSTM_PROJECTION = 1, QLSTM_PEEPHOLE = 2, QLSTM_LAYERNORM = 4, QLSTM_CIFG = 8 };

typedef enum {
    QLSTM_OK = 0,
    QLSTM_ERR_ARG = -1,       /* null pointer, bad flag combination, T or B beyond the handle's maxima */
    QLSTM_ERR_DIM = -2,       /* a dimension outside the supported range */
    QLSTM_ERR_RANGE = -3,     /* a bias with its zero-point term folded in leaves int32 (Section 6) */
    QLSTM_ERR_NOMEM = -4,     /* device or host allocation failed */
    QLSTM_ERR_CUDA = -5,      /* no device, wrong architecture, or a CUDA call failed */
    QLSTM_ERR_LAUNCH = -6,    /* the persistent kernel cannot be made co-resident on this device */
    QLSTM_ERR_TIMEOUT = -7    /* a bounded device-side wait expired; the handle stays usable */
} qlstm_error;

/* One LSTM layer: tensors and scales of Table 2.  All array pointers are HOST memory and are
 * copied by qlstm_create (the caller may free them afterwards).
 *   n_output == n_cell unless QLSTM_PROJECTION.  Each dimension <= 32768, the depth up to which
 *   an int32 accumulator of int8 products cannot overflow (Section 3.1.1); with QLSTM_LAYERNORM
 *   n_cell <= 8191 (64-bit sum of squares).
 *   With QLSTM_CIFG slot 0 (gate i) of every array must be NULL: i = min(32768 - f, 32767) (Section 3.2.9).
 *   zp_m == zp_h and eff_m targets the scale of h when there is no projection (Table 2, row m). */
typedef struct {
    int32_t n_input, n_cell, n_output;
    uint32_t flags;
    int32_t cell_int_bits;               /* m of the cell format Q_{m.15-m}, 0..15 (Section 3.2.2) */
    int32_t zp_x, zp_m, zp_h;            /* int8 zero points of input, hidden state m, output h */
    const int8_t *W[4], *R[4];           /* [n_cell][n_input], [n_cell][n_output], symmetric int8 in [-127,127] */
    const int16_t *P[4];                 /* peephole weights [n_cell] for i, f, o (slot 2 NULL); NULL unless PEEPHOLE */
    const int32_t *b[4];                 /* gate bias [n_cell]: scale s_R*s_h without LN, 2^-10*s_L with LN */
    const int16_t *L[4];                 /* layer-norm weights [n_cell]; NULL unless LAYERNORM (Section 3.2.6) */
    const int8_t *W_proj;                /* [n_output][n_cell]; NULL unless PROJECTION (Section 3.2.8) */
    const int32_t *b_proj;               /* [n_output], scale s_Wproj*s_m */
    qlstm_scale_t eff_x[4];              /* s_W s_x / s_gate      (Section 3.2.4 / 3.2.5) */
    qlstm_scale_t eff_h[4];              /* s_R s_h / s_gate */
    qlstm_scale_t eff_c[4];              /* s_P s_c / s_gate */
    qlstm_scale_t eff_ln[4];             /* 2^-10 s_L / 2^-12     (Section 3.2.6) */
    qlstm_scale_t eff_m;                 /* 2^-30 / s_m           (Section 3.2.7) */
    qlstm_scale_t eff_proj;              /* s_Wproj s_m / s_h     (Section 3.2.8) */
} qlstm_layer_t;

/*
 * qlstm_create — validates the stack, folds every zero-point term into an int32 bias
 * (Section 6: sum W (x - zp) = sum W x - zp sum W, computed in int64 and range checked),
 * repacks and uploads the weights, and allocates workspaces for sequences up to max_T steps
 * and max_B rows on CUDA device `device`.  layers[l+1].n_input must equal layers[l].n_output;
 * layer l+1 reads layer l's h with that h's zero point (layers[l+1].zp_x == layers[l].zp_h).
 * On success *out owns everything; release it with qlstm_destroy.
 */
int qlstm_create(const qlstm_layer_t *layers, int n_layers, int max_T, int max_B, int device, qlstm_t **out);

/*
 * qlstm_run — the forward pass over T steps and B independent rows (Eq. 1-7 in their integer
 * form, Section 3.2.4-3.2.9, looped over time and layers as Section 7 describes).
 *   x_dev  DEVICE int8  [T][B][n_input of layer 0]
 *   h_dev  DEVICE int8  in/out: layer after layer, [B][n_output_l]  (state h^{t-1} -> h^{T-1})
 *   c_dev  DEVICE int16 in/out: layer after layer, [B][n_cell_l]
 *   y_dev  DEVICE int8  out [T][B][n_output of the last layer]
 *   trace_dev  NULL, or DEVICE buffer of qlstm_trace_bytes() bytes receiving every intermediate
 *              tensor of every step (layout below); tracing selects slower kernels.
 *   Alignment: x_dev, c_dev, y_dev (and trace_dev) must be 16-byte aligned - the kernels read and write them with
 *              128-bit accesses and bulk copies; QLSTM_ERR_ARG otherwise.  h_dev may have any alignment.
 *   cuda_stream  a cudaStream_t (NULL = default stream).  The call only enqueues work; buffers are
 *              borrowed until that work completes.  One handle must not run concurrently with itself.
 * T == 0 or B == 0 is a no-op.  Device-side failures (QLSTM_ERR_TIMEOUT) are reported by qlstm_last_status.
 */
int qlstm_run(qlstm_t *q, const int8_t *x_dev, int T, int B, int8_t *h_dev, int16_t *c_dev,
              int8_t *y_dev, void *trace_dev, void *cuda_stream);

/* Same pass with HOST buffers: copies x, h, c to the device, runs, copies y, h, c back and
 * synchronises.  This is the end-to-end call; host buffers may be pageable or pinned. */
int qlstm_run_host(qlstm_t *q, const int8_t *x_host, int T, int B, int8_t *h_host, int16_t *c_host,
                   int8_t *y_host);

/*
 * qlstm_input_projection — step one of the pass on its own: for layer `layer`, all rows at once,
 *   X[r][g][u] = sat16(rescale(sum_j W_g[u][j] x[r][j] - zp_x sum_j W_g[u][j], eff_x[g]))   (Section 3.2.4)
 *   x_dev DEVICE int8 [rows][n_input]; out_dev DEVICE int16 [rows][n_cell][G], gates interleaved per cell: G = 4 (i, f, z, o) or 3 (f, z, o) with CIFG.
 * rows <= max_T * max_B.  x_dev must be 16-byte and out_dev 32-byte aligned (QLSTM_ERR_ARG otherwise).
 */
int qlstm_input_projection(qlstm_t *q, int layer, const int8_t *x_dev, int rows, int16_t *out_dev,
                           void *cuda_stream);

/* Synchronises the stream of the last run and returns the device-side status of that run. */
int qlstm_last_status(qlstm_t *q);

void qlstm_destroy(qlstm_t *q);
const char *qlstm_strerror(int code);

/*
 * Trace layout: for every layer (in order) and every step t one record, padded to 16 bytes:
 *   acc  int32 [4][B][C]  recurrent accumulator as fed to the rescale (bias included without LN)
 *   pacc int32 [B][O]     projection accumulator incl. bias (0 without projection)
 *   xg   int16 [4][B][C]  rescaled input contribution
 *   pre  int16 [4][B][C]  gate sum of the three rescaled terms
 *   ain  int16 [4][B][C]  input of the nonlinearity (after layer norm; = pre without it)
 *   gate int16 [4][B][C]  i, f, z, o in Q0.15
 *   c    int16 [B][C]     new cell state;   m int8 [B][C] hidden state;   h int8 [B][O] layer output
 * With CIFG slot 0 of acc / xg / pre / ain is zero and gate[0] holds the coupled input gate.
 */
size_t qlstm_trace_bytes(const qlstm_t *q, int T, int B);

/*
 * Bidirectional LSTM (Section 7: uni- and bidirectional LSTMs are loops over the same cell).  Two stacks of n_layers
 * layers read the same input: `fwd` from step 0 upwards, `bwd` from step T - 1 downwards.  Both must take the same
 * input (n_input and zp_x of their first layers equal; n_input a multiple of 16).
 *   y_dev DEVICE int8 out [T][B][O_fwd + O_bwd]: at step t the forward stack's h^t followed by the backward stack's
 *         state after it has seen x_{T-1} .. x_t.  The two halves keep their own (scale, zero point); a layer stacked on
 *         top must be quantized for an input whose two halves share one (as Table 2 does for any layer input).
 *   h_*_dev / c_*_dev DEVICE in/out state of each direction, laid out as for qlstm_run; x_dev as for qlstm_run.
 * qlstm_bidir_create takes HOST layer descriptions like qlstm_create and owns both stacks and the workspaces between
 * them; errors as for qlstm_create / qlstm_run.  qlstm_bidir_last_status synchronises and reports a device-side
 * failure of either direction.
 */
typedef struct qlstm_bidir qlstm_bidir_t;
int qlstm_bidir_create(const qlstm_layer_t *fwd_layers, const qlstm_layer_t *bwd_layers, int n_layers, int max_T, int max_B,
                       int device, qlstm_bidir_t **out);
int qlstm_bidir_run(qlstm_bidir_t *q, const int8_t *x_dev, int T, int B, int8_t *h_fwd_dev, int16_t *c_fwd_dev,
                    int8_t *h_bwd_dev, int16_t *c_bwd_dev, int8_t *y_dev, void *cuda_stream);
int qlstm_bidir_last_status(qlstm_bidir_t *q);
void qlstm_bidir_destroy(qlstm_bidir_t *q);

/*
 * qlstm_layernorm_rows_static - the integer layer norm of Section 3.2.6 (mean, variance, normalise x 2^10,
 * x L + b, rescale to Q3.12; one row = one (batch row, gate) of a step) for `rows` rows at once, for callers that
 * must not allocate.  (The paper has no counterpart: this is a packaging of its layer norm
 * for hosts where allocation is off limits - a per-frame real-time loop that cannot take the allocator's
 * device-wide lock, a process whose own arena already owns all device memory, a plug-in callback in which the
 * host forbids allocation.)
 *   q_dev DEVICE int16 [rows][n]; L_dev int16 [n]; b_dev int32 [n]; out_dev DEVICE int16 [rows][n] (Q3.12).
 *   rows <= 4096 (QLSTM_ERR_DIM beyond that: the scratch is a fixed 64 KiB array inside the library image, held
 *   by every device that loads the library until the process exits); n <= 8191.
 * It calls no cudaMalloc, cudaFree or other allocating routine.  The first call on a device looks up the
 * array's device address (with that device current) and should therefore happen before any stream capture
 * begins; later calls only launch two kernels on `cuda_stream`.  All calls share the one array and it keeps
 * whatever the last call wrote: each call overwrites every entry it later reads, so no clearing is needed, but
 * two calls that overlap on the GPU (different streams) race on it and must be serialised by the caller.
 */
int qlstm_layernorm_rows_static(const int16_t *q_dev, int rows, int n, const int16_t *L_dev, const int32_t *b_dev,
                                qlstm_scale_t eff_ln, int16_t *out_dev, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif
