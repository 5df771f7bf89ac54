/*
 * qlstm_debug.h - test, measurement and profiling hooks of libqlstm.so.
 *
 * Nothing here is needed to run the forward pass (that is include/qlstm.h).  These calls select kernel
 * families, expose host-side plans and single building blocks to the tests, exercise the bounded-wait failure
 * path without faulting the device, and read per-kernel timings.
 */
#ifndef QLSTM_DEBUG_H
#define QLSTM_DEBUG_H

#include "qlstm.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Kernel selection, for tests and measurements.  0 = automatic (default), 1 = simple kernels
 * (one thread per output, one launch per phase), 2 = fast kernels (tensor-core projection,
 * persistent recurrent kernel); 2 fails with QLSTM_ERR_DIM at run time if a shape is unsupported.
 * recurrent_impl 2 always runs layer after layer (projection launch + persistent kernel per layer), where 0 takes the
 * whole-stack kernel at small batches (up to 4 rows; up to 8 for stacks of two or more layers; up to 16 for four or more); 3 = like 2 but with the tensor-core matmuls even at batch <= 4, where 2 uses dp4a
 * mat-vecs; 4 = like 2 but with the dp4a mat-vecs up to batch 16 (the crossover is a measured default, not a limit);
 * 5 = the whole-stack kernel or QLSTM_ERR_DIM (batch > 16, or a dimension that is not a multiple of 16), with its
 * schedule chosen from the call's length; 6 = the same with the wavefront schedule (one group of blocks per layer)
 * forced, 7 = with the sequential schedule (every layer on all blocks) forced. */
int qlstm_set_impl(qlstm_t *q, int projection_impl, int recurrent_impl);

/* Failure-path check: with missing_arrivals > 0 every grid barrier of the persistent recurrent kernel (and every
 * counter wait of the whole-stack kernel) waits for
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
/*
 * The persistent recurrent kernel memoises the nonlinearities of Section 3.2.1: at qlstm_create the definition is
 * evaluated once over the whole int16 domain and packed into per-layer tables (plain uint16, or one 32-bit word per four
 * inputs), which the kernel copies into shared memory before every elementwise phase.
 *   qlstm_eval_activation_tables builds the tables of a layer whose cell state has cell_int_bits integer bits exactly as
 *     qlstm_create does for a kernel with max_bytes (<= 131072) of idle shared memory, and looks every int16 input up with
 *     the kernel's own lookup code: sigmoid_dev (Q3.12 in), tanh_gate_dev (Q3.12 in), tanh_cell_dev (Q_{m.15-m} in,
 *     m = cell_int_bits): DEVICE int16 [65536], entry x + 32768.  layout_out7 (HOST) = { bytes of the tables, byte offset
 *     of the gate tanh, of the cell tanh, last |x| with an entry of its own for the two, format of the cell tanh
 *     (0 shared with the gate's, 1 packed, 2 plain), format of the sigmoid (0 plain, 1 packed) }; bytes = 0 means that
 *     the tables do not fit or that the definition failed a check the formats rely on (the outputs are then untouched;
 *     such a layer keeps the arithmetic).  Synchronises the stream.
 *   qlstm_debug_activation_tables(q, 0) makes the kernel evaluate the definition instead (1 restores the default); 2
 *     selects the kernel's general instantiation, the one a layer gets when one of its scales has a left shift
 *     (shift > 0), which otherwise only such layers reach.  Returns the number of layers that hold tables, or a
 *     negative qlstm_error.
 */
int qlstm_eval_activation_tables(int cell_int_bits, int max_bytes, int16_t *sigmoid_dev, int16_t *tanh_gate_dev,
                                 int16_t *tanh_cell_dev, int *layout_out7, void *cuda_stream);
int qlstm_debug_activation_tables(qlstm_t *q, int enable);
int qlstm_eval_layernorm_row(const int16_t *q_dev, int n, const int16_t *L_dev, const int32_t *b_dev,
                             qlstm_scale_t eff_ln, int16_t *out_dev, void *cuda_stream);

/* Two measurements the roofline statements rest on, each a kernel of its own on device `device` (no handle needed).
 *   qlstm_debug_mma_i8_peak: every SM issues `iters` x 4 back-to-back tcgen05.mma kind::i8 (M128 N256 K32) from
 *     operands resident in shared memory; *tops_out = achieved int8 TOP/s (best of three timed launches).  This is the
 *     measured issue-rate peak of the tensor path that the input projection of Section 3.2.4 runs on.
 *   qlstm_debug_barrier_latency: n_barriers grid-wide barriers of the persistent kernel's kind back to back on one
 *     block per SM; *us_per_barrier_out = microseconds per barrier (the floor of every phase boundary of a time step).
 * QLSTM_ERR_ARG on bad arguments, QLSTM_ERR_TIMEOUT if a (bounded) wait inside the kernel ran out. */
int qlstm_debug_mma_i8_peak(int device, int iters, double *tops_out);
int qlstm_debug_barrier_latency(int device, int n_barriers, double *us_per_barrier_out);

/* Device properties the library sees: SM count, and resident blocks of the persistent kernel. */
int qlstm_device_info(qlstm_t *q, int *sm_count, int *persistent_blocks);

#ifdef __cplusplus
}
#endif
#endif
