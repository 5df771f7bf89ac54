/*
 * qlstm_calib.h - the steps before the integer path, on the GPU: post-training statistics collection (Section 4) and
 * the quantization recipe of Table 2.
 *
 * qlstm_calibrate runs the float LSTM of Eq. 1-7 (fp64, every variant of Section 2) over a calibration batch on the
 * device and logs the range of every tensor whose scale Table 2 derives from measurement: layer input x, output h,
 * hidden state m (min / max), cell state c (max |.|), and with layer norm the gate sums before normalisation
 * (max |.| per gate, Section 3.2.5).  qlstm_quantize_model applies Table 2: the reductions over the weights
 * (max |.| per tensor) and the rounding of weights and biases run on the device; the handful of scalars that follow
 * (scales, zero points, the cell format, effective scales encoded as (multiplier, shift)) are computed on the host.
 * The result holds HOST tensors in the form qlstm_create takes.
 *
 * Conventions as in qlstm.h: gate order i, f, z, o; matrices row-major [output unit][input unit]; with QLSTM_CIFG
 * slot 0 of every array is NULL.  Every call returns 0 or a negative qlstm_error.
 */
#ifndef QLSTM_CALIB_H
#define QLSTM_CALIB_H

#include "qlstm.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Float parameters of one layer (HOST pointers, fp64). */
typedef struct {
    int32_t n_input, n_cell, n_output;
    uint32_t flags;                       /* QLSTM_PROJECTION | QLSTM_PEEPHOLE | QLSTM_LAYERNORM | QLSTM_CIFG */
    const double *W[4], *R[4];            /* [n_cell][n_input], [n_cell][n_output] */
    const double *P[4];                   /* peephole [n_cell] for i, f, o (slot 2 NULL); NULL unless PEEPHOLE */
    const double *L[4];                   /* layer-norm weights [n_cell]; NULL unless LAYERNORM */
    const double *b[4];                   /* gate bias [n_cell] */
    const double *W_proj, *b_proj;        /* [n_output][n_cell], [n_output]; NULL unless PROJECTION */
} qlstm_float_layer_t;

/* Ranges logged during the float run (the "log" nodes of the paper's training-graph figures). */
typedef struct {
    double x_min, x_max;                  /* layer input over all steps and rows */
    double h_min, h_max;                  /* layer output, the initial state 0 included */
    double m_min, m_max;                  /* hidden state before the projection */
    double c_absmax;                      /* cell state */
    double g_absmax[4];                   /* layer norm only: gate sums before normalisation, per gate */
} qlstm_ranges_t;

/*
 * qlstm_calibrate - float forward pass of the stack over x_host [T][B][n_input of layer 0] (HOST, fp64) on CUDA
 * device `device`, initial h = 0 and c = 0; ranges_out (HOST) receives one entry per layer.
 */
int qlstm_calibrate(const qlstm_float_layer_t *layers, int n_layers, const double *x_host, int T, int B, int device,
                    qlstm_ranges_t *ranges_out);

/*
 * qlstm_quantize_model - Table 2 applied to the stack with the logged ranges: int8 weights (scale max|W| / 127), int16
 * peephole and layer-norm weights (max|.| / 32767), int32 biases (scale s_R s_h without layer norm, 2^-10 s_L with it),
 * int8 asymmetric x / h / m (range widened to contain 0, / 255, zero point rounded and clamped), power-of-two cell
 * range Q_{m.15-m}, effective scales as (multiplier, shift).  Layer l + 1 reads layer l's h with that h's scale and
 * zero point.  *out owns every tensor; release it with qlstm_quantized_destroy.
 */
typedef struct qlstm_quantized qlstm_quantized_t;
int qlstm_quantize_model(const qlstm_float_layer_t *layers, const qlstm_ranges_t *ranges, int n_layers, int device,
                         qlstm_quantized_t **out);
/* The quantized stack as qlstm_create takes it (HOST pointers owned by q). */
const qlstm_layer_t *qlstm_quantized_layers(const qlstm_quantized_t *q);
/* Real scales of layer `layer` for de-quantizing: out4 = { s_x, s_h, s_m, s_c }. */
int qlstm_quantized_scales(const qlstm_quantized_t *q, int layer, double *out4);
void qlstm_quantized_destroy(qlstm_quantized_t *q);

#ifdef __cplusplus
}
#endif
#endif
