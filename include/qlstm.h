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
 * rows <= max_T * max_B.
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

/* Kernel selection, for tests and measurements.  0 = automatic (default), 1 = simple kernels
 * (one thread per output, one launch per phase), 2 = fast kernels (tensor-core projection,
 * persistent recurrent kernel); 2 fails with QLSTM_ERR_DIM at run time if a shape is unsupported.
 * recurrent_impl 3 = like 2 but with the tensor-core matmuls even at batch <= 4, where 0 and 2 use dp4a mat-vecs;
 * 4 = like 2 but with the dp4a mat-vecs up to batch 16 (the crossover is a measured default, not a limit). */
int qlstm_set_impl(qlstm_t *q, int projection_impl, int recurrent_impl);

/* Failure-path check: with missing_arrivals > 0 every grid barrier of the persistent recurrent kernel waits for
 * that many arrivals that never come, for at most limit_ns (<= 1 s); the wait then runs out, the kernel sets its
 * status word, every block leaves the time loop, frees its tensor memory and returns, and qlstm_last_status
 * reports QLSTM_ERR_TIMEOUT.  Nothing faults or hangs and the handle stays usable; 0 restores normal operation. */
int qlstm_debug_barrier_timeout(qlstm_t *q, int missing_arrivals, unsigned long long limit_ns);

/* Host logic of the persistent kernel's operand ring, exposed for tests (no device is touched).  The matmuls of
 * Section 3.2.4 / 3.2.8 stream their batch operand through `stages` ring stages that one producer fills and
 * `n_owners` MMA issuers drain; within a phase owner o uses the stages o, o + n_owners, ... only, so that no
 * thread ever waits for a round of a stage whose previous round it did not consume itself.
 * contiguous != 0: one operand tile of chunks_per_tile chunks per owner; else chunks_total chunks of one tile dealt
 * round-robin.  out14 (host) receives n_owners, the largest chunk count of an owner, chunks[4] and stages[4] per
 * owner, and the fills of each of the 4 stages in the phase.  QLSTM_ERR_ARG unless 1 <= n_owners <= stages <= 4. */
int qlstm_debug_ring_plan(int stages, int n_owners, int contiguous, int chunks_per_tile, int chunks_total, int *out14);

/* Host logic of the input-projection kernel's tiling (Section 3.2.4, first rescale term), exposed for tests (no
 * device is touched).  For a handle created for max_rows = max_T x max_B rows, a projection of rows <= max_rows rows
 * onto n_gate_rows = cells x gates outputs with n_input columns, on a device of sm_count SMs with smem_bytes of
 * shared memory per block: out5 (host) receives the panel width (gate rows of W resident per block; fixed at create
 * time from max_rows), the depth of the x ring, the output tiles per block, the number of m-tile ranges (> 0: block b
 * keeps panel b % panels and walks range b / panels; 0: equal contiguous ranges of the panel-major tile numbering)
 * and the grid size.  QLSTM_ERR_ARG on a non-positive argument, rows > max_rows or NULL; QLSTM_ERR_DIM when no panel
 * of these shapes fits in shared memory (such layers take the simple kernel). */
int qlstm_debug_projection_plan(long long max_rows, long long rows, int n_gate_rows, int n_input, int sm_count,
                                int smem_bytes, int *out5);

/* Per-kernel device times of the runs since the last reset, measured with CUDA events on the
 * run's stream when profiling is on (it adds two event records per launch).
 * qlstm_set_profiling levels: 0 off; 1 the per-kernel event times; 2 also the device phase timers inside the
 * persistent recurrent kernel.  Level 2 perturbs what it measures (the first block updates its timers in
 * global memory before every grid barrier and so arrives late at each), so take throughput numbers at
 * level 0 or 1 and the phase breakdown in a separate pass. */
typedef struct {
    double projection_ms; int projection_launches;
    double recurrent_ms;  int recurrent_launches;
    double other_ms;      int other_launches;
    /* inside the persistent recurrent kernel, as seen by its first block (device timer): time spent working in
     * the matmul (a), elementwise (b) and projection (c) phases, and waiting at the grid barrier after each */
    double phase_a_ms, wait_a_ms, phase_b_ms, wait_b_ms, phase_c_ms, wait_c_ms;
    double matmul_a_ms;   /* part of phase_a_ms before the first accumulator is ready (operand load + MMA) */
} qlstm_profile_t;
int qlstm_set_profiling(qlstm_t *q, int level);
int qlstm_get_profile(qlstm_t *q, qlstm_profile_t *out, int reset);

/*
 * Evaluators of two building blocks on their own, on the current device, with the same device code the
 * recurrent kernel runs.  They exist so that the integer nonlinearities can be checked over their whole
 * domain (Section 3.2.1: int16 Q_{m.15-m} in, Q0.15 out) and the integer layer norm (Section 3.2.6) on
 * hand-picked rows.
 *   qlstm_eval_activations: sigmoid_dev / tanh_dev DEVICE int16 [65536], entry x + 32768 holds f(x) for the
 *     input format Q_{m.15-m} with m = cell_int_bits (gates use m = 3).
 *   qlstm_eval_layernorm_row: q_dev int16 [n], L_dev int16 [n], b_dev int32 [n], out_dev int16 [n] (Q3.12);
 *     n <= 8191.
 */
int qlstm_eval_activations(int cell_int_bits, int16_t *sigmoid_dev, int16_t *tanh_dev, void *cuda_stream);
int qlstm_eval_layernorm_row(const int16_t *q_dev, int n, const int16_t *L_dev, const int32_t *b_dev,
                             qlstm_scale_t eff_ln, int16_t *out_dev, void *cuda_stream);

/*
 * qlstm_layernorm_rows_static - the integer layer norm of qlstm_eval_layernorm_row for `rows` rows at once,
 * for callers that must not allocate.  (The paper has no counterpart: this is a packaging of its layer norm
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

/* Device properties the library sees: SM count, and resident blocks of the persistent kernel. */
int qlstm_device_info(qlstm_t *q, int *sm_count, int *persistent_blocks);

#ifdef __cplusplus
}
#endif
#endif
