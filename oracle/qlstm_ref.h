/*
 * CPU oracle of the integer-only LSTM forward pass ("On the quantization of
 * recurrent neural networks", Section 3 and Section 6).
 *
 * TEST INFRASTRUCTURE ONLY.  This library defines the expected result of the
 * integer execution graph in plain, slow, sequential C.  Tests, the smoke
 * check and the benchmark's CPU-baseline leg call it; no product path does.
 * It shares no source, header, table or helper with the CUDA implementation.
 *
 * Conventions (readings of the paper, all restated in the project's design notes):
 *   - affine quantization real = scale * (q - zero_point); matmuls use (q - zp),
 *     a requantize step adds the output zero point;
 *   - every "round", "rescale" and "shift" rounds to nearest, ties away from zero;
 *   - gate order i, f, z, o; matrices row-major [output unit][input unit];
 *   - a real effective scale is multiplier * 2^(shift - 31), multiplier in [2^30, 2^31) or 0.
 *
 * Pins (tests/test_oracle_*.py): exhaustive int16 sweeps of the integer sigmoid / tanh
 * against fp64 closed forms, exact rational arithmetic for the rescale, brute-force
 * square roots, the paper's printed values, the zero-point identity, agreement with
 * an independent NumPy restatement, and agreement with the fp64 LSTM of Eq. 1-7.
 * Parity with any deployed runtime is unpinned (none exists in this project) and not a goal.
 */
#ifndef QLSTM_REF_H
#define QLSTM_REF_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct { int32_t multiplier; int32_t shift; } qref_scale;

enum { QREF_PROJECTION = 1, QREF_PEEPHOLE = 2, QREF_LAYERNORM = 4, QREF_CIFG = 8 };

typedef struct {
    int32_t n_input, n_cell, n_output;
    uint32_t flags;
    int32_t cell_int_bits;               /* m of Q_{m.15-m} (Section 3.2.2) */
    int32_t zp_x, zp_m, zp_h;
    const int8_t *W[4], *R[4];           /* [n_cell][n_input], [n_cell][n_output]; slot 0 NULL with CIFG */
    const int16_t *P[4];                 /* peephole weights [n_cell] for i, f, o */
    const int32_t *b[4];                 /* gate bias [n_cell] */
    const int16_t *L[4];                 /* layer-norm weights [n_cell] */
    const int8_t *W_proj;                /* [n_output][n_cell] */
    const int32_t *b_proj;               /* [n_output] */
    qref_scale eff_x[4], eff_h[4], eff_c[4], eff_ln[4], eff_m, eff_proj;
} qref_layer;

/* Fixed-point primitives the paper names but does not define ("rescale", "shift"). */
int32_t qref_srdhm(int32_t a, int32_t b);           /* saturating rounding doubling high multiply */
int64_t qref_rdivpot(int64_t x, int e);             /* x / 2^e, ties away from zero, e >= 0 */
int32_t qref_mbqm(int32_t x, qref_scale s);         /* x * multiplier * 2^(shift-31) */
int64_t qref_rdiv(int64_t n, int64_t d);            /* n / d, d > 0, ties away from zero */
uint64_t qref_isqrt(uint64_t v);                    /* floor(sqrt(v)) */

/* Integer sigmoid / tanh: int16 Q_{m.15-m} in, Q_{0.15} out (Section 3.2.1). */
int16_t qref_sigmoid(int16_t x, int m);
int16_t qref_tanh(int16_t x, int m);

/* Integer layer normalisation of one row (Section 3.2.6, Eq. 13-16). */
void qref_layernorm_row(const int16_t *q, int n, const int16_t *L, const int32_t *b,
                        qref_scale eff_ln, int16_t *out);

/* Bytes of the per-timestep trace for a run (see qlstm_ref.c for the record layout). */
size_t qref_trace_bytes(const qref_layer *layers, int n_layers, int T, int B);

/*
 * Runs the whole stack over T steps for B independent rows, all pointers HOST memory.
 *   x [T][B][I0] int8; h [sum_l B*O_l] int8 in/out; c [sum_l B*C_l] int16 in/out;
 *   y [T][B][O_last] int8 out; trace NULL or qref_trace_bytes() bytes.
 * Returns 0, or -1 on an invalid argument.
 */
int qref_run(const qref_layer *layers, int n_layers, const int8_t *x, int T, int B,
             int8_t *h, int16_t *c, int8_t *y, void *trace);

int qref_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
