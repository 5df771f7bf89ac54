/*
 * CPU oracle of the integer-only LSTM forward pass.  TEST INFRASTRUCTURE ONLY:
 * see qlstm_ref.h for what it is, what pins it and who may call it.
 *
 * The code follows the paper's integer execution formulas in the paper's order:
 *   gate sums (Section 3.2.4 / 3.2.5) -> integer layer norm (Section 3.2.6, Eq. 13-16)
 *   -> integer sigmoid / tanh (Section 3.2.1) -> CIFG coupling (Section 3.2.9)
 *   -> cell update and hidden state (Section 3.2.7) -> projection (Section 3.2.8),
 * looped over time and layers (Section 7).  Zero points are subtracted inside the
 * matmuls (the unfolded form of Section 6), so that the folded form of the CUDA
 * path is checked against the definition rather than against itself.
 *
 * No blocking, fusion or reordering: one (layer, t, batch row) at a time.  Batch rows
 * never interact (Eq. 1-7 are per example, layer norm is per row), so the loop over
 * rows may run on several threads without changing any result.
 */
#include "qlstm_ref.h"

#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------------------------------------------------------------- primitives */

static inline int32_t sat32(int64_t v)
{
    return v > INT32_MAX ? INT32_MAX : (v < INT32_MIN ? INT32_MIN : (int32_t)v);
}
static inline int16_t sat16(int64_t v)
{
    return v > 32767 ? 32767 : (v < -32768 ? -32768 : (int16_t)v);
}
static inline int8_t sat8(int64_t v)
{
    return v > 127 ? 127 : (v < -128 ? -128 : (int8_t)v);
}

/* x / 2^e rounded to nearest, ties away from zero ("shift" of Section 3.2.7). |x| < 2^62. */
int64_t qref_rdivpot(int64_t x, int e)
{
    if (e <= 0) return x;
    if (e > 62) return 0;
    int64_t ax = x < 0 ? -x : x;
    int64_t q = (ax + ((int64_t)1 << (e - 1))) >> e;
    return x < 0 ? -q : q;
}

/* round(a * b / 2^31), ties away from zero; the one overflowing case saturates. */
int32_t qref_srdhm(int32_t a, int32_t b)
{
    if (a == INT32_MIN && b == INT32_MIN) return INT32_MAX;
    int64_t p = (int64_t)a * (int64_t)b;
    int64_t ap = p < 0 ? -p : p;
    int64_t q = (ap + ((int64_t)1 << 30)) >> 31;
    return (int32_t)(p < 0 ? -q : q);
}

/* "rescale" of the execution formulas: x times the real scale multiplier * 2^(shift-31).
 * A positive shift is applied first, as a saturating left shift. */
int32_t qref_mbqm(int32_t x, qref_scale s)
{
    int left = s.shift > 0 ? s.shift : 0;
    int right = s.shift < 0 ? -s.shift : 0;
    int32_t xl = sat32((int64_t)x * ((int64_t)1 << left));
    return (int32_t)qref_rdivpot(qref_srdhm(xl, s.multiplier), right);
}

/* n / d for d > 0, rounded to nearest, ties away from zero. |n| < 2^63 - d. */
int64_t qref_rdiv(int64_t n, int64_t d)
{
    uint64_t an = n < 0 ? (uint64_t)0 - (uint64_t)n : (uint64_t)n;
    uint64_t q = (an + ((uint64_t)d >> 1)) / (uint64_t)d;
    return n < 0 ? -(int64_t)q : (int64_t)q;
}

/* floor(sqrt(v)), digit by digit. */
uint64_t qref_isqrt(uint64_t v)
{
    uint64_t r = 0, bit = (uint64_t)1 << 62;
    while (bit > v) bit >>= 2;
    while (bit) {
        if (v >= r + bit) { v -= r + bit; r = (r >> 1) + bit; }
        else r >>= 1;
        bit >>= 2;
    }
    return r;
}

/* ------------------------------------------------- integer sigmoid and tanh
 *
 * The paper fixes the formats (int16 Q_{m.15-m} in, Q_{0.15} out, output clamped to
 * [-1, 32767/32768], no lookup table, no inner branch, no float) but not the algorithm.
 * Definition used here, for |x| and then mirrored:
 *   exp(-k|x|) = 2^(-t),  t = k |x| log2(e) in Q26,  k = 1 (sigmoid) or 2 (tanh);
 *   2^(-t) = 2^(-n) * 2^(-f), n = integer part, f = fraction; 2^(-f) by a degree-6
 *   Taylor polynomial around f = 1/2 evaluated in Q30; E ~ 2^30 exp(-k|x|);
 *   sigmoid(|x|) = 2^30 / (2^30 + E),  tanh(|x|) = (2^30 - E) / (2^30 + E),
 *   each one exact integer division rounded half up to Q0.15.
 * Constants: LOG2E_Q30 = round(2^30 log2 e); POLY[k] = round(2^30 2^(-1/2) (-ln 2)^k / k!).
 */
static const int64_t LOG2E_Q30 = 1549082005;
static const int64_t POLY[7] = { 759250125, -526272083, 182392005, -42141501, 7302566, -1012351, 116951 };

/* E = round(2^30 * exp(-k * |x| * 2^-(15-m))), k in {1, 2}; 0 <= E <= about 2^30. */
static int64_t exp_neg_q30(int32_t absx, int m, int k)
{
    int frac_bits = 15 - m;
    int64_t t = qref_rdivpot((int64_t)absx * LOG2E_Q30 * k, frac_bits + 4); /* Q26 */
    int64_t n = t >> 26;
    if (n > 40) n = 40;
    int64_t f = t & (((int64_t)1 << 26) - 1);
    int64_t g = f - ((int64_t)1 << 25);
    int64_t acc = POLY[6];
    for (int i = 5; i >= 0; --i) acc = qref_rdivpot(acc * g, 26) + POLY[i];
    return qref_rdivpot(acc, (int)n);
}

int16_t qref_sigmoid(int16_t x, int m)
{
    int32_t a = x < 0 ? -(int32_t)x : (int32_t)x;
    int64_t E = exp_neg_q30(a, m, 1);
    int64_t D = ((int64_t)1 << 30) + E;
    int64_t S = (((int64_t)1 << 46) + D) / (2 * D);        /* round-half-up of 2^45 / D */
    if (x >= 0) return (int16_t)(S > 32767 ? 32767 : S);
    return (int16_t)(32768 - S);
}

int16_t qref_tanh(int16_t x, int m)
{
    int32_t a = x < 0 ? -(int32_t)x : (int32_t)x;
    int64_t E = exp_neg_q30(a, m, 2);
    int64_t D = ((int64_t)1 << 30) + E;
    int64_t N = ((int64_t)1 << 30) - E;
    int64_t Tq = (2 * N * 32768 + D) / (2 * D);            /* round-half-up of 2^15 N / D */
    if (x >= 0) return (int16_t)(Tq > 32767 ? 32767 : Tq);
    return (int16_t)(-Tq);
}

/* ------------------------------------------------- integer layer normalisation
 *
 * Section 3.2.6 with s' = 2^-10:
 *   mean   = round(2^10 * sum(q) / n)
 *   var    = round(2^20 * sum(q^2) / n) - mean^2,   sigma = floor(sqrt(max(var, 0)))
 *   q'_i   = round(2^10 * (2^10 q_i - mean) / sigma)        (0 for the whole row if sigma = 0)
 *   out_i  = sat16(rescale(sat32(q'_i * L_i + b_i), eff_ln))   -> Q3.12
 * The second factor 2^10 in q' is the "x 2^10" node of the layer-norm execution figure: it
 * puts q' at scale 2^-10, the scale the bias (2^-10 * s_L) is quantized with.
 */
void qref_layernorm_row(const int16_t *q, int n, const int16_t *L, const int32_t *b,
                        qref_scale eff_ln, int16_t *out)
{
    int64_t sum = 0, sumsq = 0;
    for (int i = 0; i < n; ++i) { sum += q[i]; sumsq += (int64_t)q[i] * q[i]; }
    int64_t mean = qref_rdiv(sum * 1024, n);
    int64_t var = qref_rdiv(sumsq * 1048576, n) - mean * mean;
    int64_t sigma = (int64_t)qref_isqrt(var > 0 ? (uint64_t)var : 0);
    for (int i = 0; i < n; ++i) {
        int64_t qp = sigma == 0 ? 0 : qref_rdiv(1024 * (1024 * (int64_t)q[i] - mean), sigma);
        int64_t v = qp * (int64_t)L[i] + (int64_t)b[i];
        out[i] = sat16(qref_mbqm(sat32(v), eff_ln));
    }
}

/* ------------------------------------------------- trace layout
 *
 * For every layer (in order) and every step t one record, 16-byte aligned:
 *   acc  int32 [4][B][C]  recurrent accumulator as fed to the rescale (bias included without LN)
 *   pacc int32 [B][O]     projection accumulator incl. bias (0 without projection)
 *   xg   int16 [4][B][C]  rescaled input contribution  rescale(W (x - zp), eff_x)
 *   pre  int16 [4][B][C]  gate sum of the three rescaled terms
 *   ain  int16 [4][B][C]  input of the nonlinearity (after layer norm; = pre without it)
 *   gate int16 [4][B][C]  i, f, z, o in Q0.15
 *   c    int16 [B][C]     new cell state
 *   m    int8  [B][C]     hidden state before projection
 *   h    int8  [B][O]     layer output
 * With CIFG slot 0 of acc / xg / pre / ain is zero and gate[0] holds the coupled input gate.
 */
static size_t record_bytes(const qref_layer *l, int B)
{
    size_t bc = (size_t)B * l->n_cell, bo = (size_t)B * l->n_output;
    size_t n = 4 * (4 * bc) + 4 * bo + 2 * (4 * bc) * 4 + 2 * bc + bc + bo;
    return (n + 15) & ~(size_t)15;
}

size_t qref_trace_bytes(const qref_layer *layers, int n_layers, int T, int B)
{
    size_t total = 0;
    for (int l = 0; l < n_layers; ++l) total += (size_t)T * record_bytes(&layers[l], B);
    return total;
}

typedef struct {
    int32_t *acc, *pacc;
    int16_t *xg, *pre, *ain, *gate, *c;
    int8_t *m, *h;
} record_view;

static record_view view_record(uint8_t *p, const qref_layer *l, int B)
{
    size_t bc = (size_t)B * l->n_cell, bo = (size_t)B * l->n_output;
    record_view v;
    v.acc = (int32_t *)p;            p += 4 * 4 * bc;
    v.pacc = (int32_t *)p;           p += 4 * bo;
    v.xg = (int16_t *)p;             p += 2 * 4 * bc;
    v.pre = (int16_t *)p;            p += 2 * 4 * bc;
    v.ain = (int16_t *)p;            p += 2 * 4 * bc;
    v.gate = (int16_t *)p;           p += 2 * 4 * bc;
    v.c = (int16_t *)p;              p += 2 * bc;
    v.m = (int8_t *)p;               p += bc;
    v.h = (int8_t *)p;
    return v;
}

/* ------------------------------------------------- one cell step for one batch row */

typedef struct {
    int32_t *acc;     /* [4][C] */
    int32_t *pacc;    /* [O]    */
    int16_t *xg, *pre, *ain, *gate;   /* [4][C] each */
    int8_t *m;        /* [C] */
} row_scratch;

/* sum_k w[k] * (a[k] - zp).  |w (a - zp)| <= 127 * 255 and n <= 2^15, so the sum stays
 * below 2^31 and an int32 accumulator is exact (the overflow bound of Section 3.1.1). */
static int32_t dot_i8(const int8_t *w, const int8_t *a, int32_t zp, int n)
{
    int32_t acc = 0;
    for (int k = 0; k < n; ++k) acc += (int32_t)w[k] * ((int32_t)a[k] - zp);
    return acc;
}

/* gate sum of Section 3.2.4 / 3.2.5 for gate g, all cells: three rescaled terms added. */
static void gate_sum(const qref_layer *l, int g, const int8_t *x, const int8_t *h,
                     const int16_t *c_peep, row_scratch *s)
{
    const int C = l->n_cell, I = l->n_input, O = l->n_output;
    const int ln = (l->flags & QREF_LAYERNORM) != 0;
    for (int u = 0; u < C; ++u) {
        int32_t ax = dot_i8(&l->W[g][(size_t)u * I], x, l->zp_x, I);
        int16_t X = sat16(qref_mbqm(ax, l->eff_x[g]));

        int64_t ah = dot_i8(&l->R[g][(size_t)u * O], h, l->zp_h, O);
        if (!ln) ah += l->b[g][u];                 /* bias rides on the recurrent accumulator */
        int32_t A = sat32(ah);
        int16_t H = sat16(qref_mbqm(A, l->eff_h[g]));

        int16_t Pc = 0;
        if ((l->flags & QREF_PEEPHOLE) && c_peep != NULL)
            Pc = sat16(qref_mbqm((int32_t)l->P[g][u] * (int32_t)c_peep[u], l->eff_c[g]));

        s->acc[g * C + u] = A;
        s->xg[g * C + u] = X;
        s->pre[g * C + u] = sat16((int32_t)X + (int32_t)H + (int32_t)Pc);
    }
    if (ln)
        qref_layernorm_row(&s->pre[g * C], C, l->L[g], l->b[g], l->eff_ln[g], &s->ain[g * C]);
    else
        memcpy(&s->ain[g * C], &s->pre[g * C], sizeof(int16_t) * C);
}

static void step_row(const qref_layer *l, const int8_t *x, int8_t *h, int16_t *c, row_scratch *s)
{
    const int C = l->n_cell, O = l->n_output, m = l->cell_int_bits;
    const int cifg = (l->flags & QREF_CIFG) != 0;
    int16_t *gi = &s->gate[0 * C], *gf = &s->gate[1 * C], *gz = &s->gate[2 * C], *go = &s->gate[3 * C];

    /* forget, input and update gates see c^{t-1} (Eq. 1-3) */
    gate_sum(l, 1, x, h, c, s);
    for (int u = 0; u < C; ++u) gf[u] = qref_sigmoid(s->ain[1 * C + u], 3);
    if (cifg) {
        for (int u = 0; u < C; ++u) {
            int32_t v = 32768 - (int32_t)gf[u];            /* 1 - f in Q0.15, Section 3.2.9 */
            gi[u] = (int16_t)(v > 32767 ? 32767 : v);
            s->acc[u] = 0; s->xg[u] = 0; s->pre[u] = 0; s->ain[u] = 0;
        }
    } else {
        gate_sum(l, 0, x, h, c, s);
        for (int u = 0; u < C; ++u) gi[u] = qref_sigmoid(s->ain[0 * C + u], 3);
    }
    gate_sum(l, 2, x, h, NULL, s);
    for (int u = 0; u < C; ++u) gz[u] = qref_tanh(s->ain[2 * C + u], 3);

    /* cell update, Eq. 4: Q0.15 * Q0.15 -> Q_{m.15-m} is a shift by 15 + m, Q0.15 * Q_{m.15-m} by 15 */
    for (int u = 0; u < C; ++u) {
        int64_t iz = qref_rdivpot((int32_t)gi[u] * (int32_t)gz[u], 15 + m);
        int64_t fc = qref_rdivpot((int32_t)gf[u] * (int32_t)c[u], 15);
        c[u] = sat16(iz + fc);
    }

    /* output gate sees the new cell state (Eq. 5) */
    gate_sum(l, 3, x, h, c, s);
    for (int u = 0; u < C; ++u) go[u] = qref_sigmoid(s->ain[3 * C + u], 3);

    /* hidden state, Eq. 6: tanh takes the cell's own Q_{m.15-m} format */
    for (int u = 0; u < C; ++u) {
        int32_t prod = (int32_t)go[u] * (int32_t)qref_tanh(c[u], m);
        s->m[u] = sat8((int64_t)qref_mbqm(prod, l->eff_m) + l->zp_m);
    }

    /* projection, Eq. 7 */
    if (l->flags & QREF_PROJECTION) {
        for (int p = 0; p < O; ++p) {
            int64_t a = (int64_t)dot_i8(&l->W_proj[(size_t)p * C], s->m, l->zp_m, C) + l->b_proj[p];
            s->pacc[p] = sat32(a);
            h[p] = sat8((int64_t)qref_mbqm(s->pacc[p], l->eff_proj) + l->zp_h);
        }
    } else {
        for (int p = 0; p < O; ++p) { s->pacc[p] = 0; h[p] = s->m[p]; }
    }
}

/* ------------------------------------------------- sequence and layer loops */

static int layer_ok(const qref_layer *l)
{
    if (l->n_input <= 0 || l->n_cell <= 0 || l->n_output <= 0) return 0;
    if (l->n_input > 32768 || l->n_cell > 32768 || l->n_output > 32768) return 0;   /* Section 3.1.1 */
    if (!(l->flags & QREF_PROJECTION) && l->n_output != l->n_cell) return 0;
    if ((l->flags & QREF_LAYERNORM) && l->n_cell > 8191) return 0;
    if (l->cell_int_bits < 0 || l->cell_int_bits > 15) return 0;
    return 1;
}

int qref_run(const qref_layer *layers, int n_layers, const int8_t *x, int T, int B,
             int8_t *h, int16_t *c, int8_t *y, void *trace)
{
    if (!layers || n_layers <= 0 || !x || T < 0 || B < 0 || !h || !c || !y) return -1;
    for (int l = 0; l < n_layers; ++l) {
        if (!layer_ok(&layers[l])) return -1;
        if (l > 0 && layers[l].n_input != layers[l - 1].n_output) return -1;
    }
    if (T == 0 || B == 0) return 0;

    int max_o = 0;
    for (int l = 0; l < n_layers; ++l) if (layers[l].n_output > max_o) max_o = layers[l].n_output;
    /* two ping-pong buffers hold the sequences passed between layers */
    int8_t *seq[2] = { NULL, NULL };
    if (n_layers > 1) {
        seq[0] = (int8_t *)malloc((size_t)T * B * max_o);
        seq[1] = (int8_t *)malloc((size_t)T * B * max_o);
        if (!seq[0] || !seq[1]) { free(seq[0]); free(seq[1]); return -1; }
    }

    const int8_t *in = x;
    size_t h_off = 0, c_off = 0;
    uint8_t *tr = (uint8_t *)trace;
    for (int li = 0; li < n_layers; ++li) {
        const qref_layer *l = &layers[li];
        const int C = l->n_cell, O = l->n_output, I = l->n_input;
        int8_t *out = (li == n_layers - 1) ? y : seq[li & 1];
        int8_t *hl = h + h_off;
        int16_t *cl = c + c_off;
        size_t rec = record_bytes(l, B);

        #pragma omp parallel
        {
            row_scratch s;
            s.acc = (int32_t *)malloc(sizeof(int32_t) * 4 * C);
            s.pacc = (int32_t *)malloc(sizeof(int32_t) * O);
            s.xg = (int16_t *)malloc(sizeof(int16_t) * 4 * C);
            s.pre = (int16_t *)malloc(sizeof(int16_t) * 4 * C);
            s.ain = (int16_t *)malloc(sizeof(int16_t) * 4 * C);
            s.gate = (int16_t *)malloc(sizeof(int16_t) * 4 * C);
            s.m = (int8_t *)malloc(C);
            /* rows are independent: each thread walks its rows through all T steps */
            #pragma omp for schedule(static)
            for (int b = 0; b < B; ++b) {
                for (int t = 0; t < T; ++t) {
                    const int8_t *xr = in + ((size_t)t * B + b) * I;
                    step_row(l, xr, hl + (size_t)b * O, cl + (size_t)b * C, &s);
                    memcpy(out + ((size_t)t * B + b) * O, hl + (size_t)b * O, O);
                    if (tr) {
                        record_view v = view_record(tr + (size_t)t * rec, l, B);
                        for (int g = 0; g < 4; ++g) {
                            size_t o = ((size_t)g * B + b) * C;
                            memcpy(v.acc + o, s.acc + g * C, sizeof(int32_t) * C);
                            memcpy(v.xg + o, s.xg + g * C, sizeof(int16_t) * C);
                            memcpy(v.pre + o, s.pre + g * C, sizeof(int16_t) * C);
                            memcpy(v.ain + o, s.ain + g * C, sizeof(int16_t) * C);
                            memcpy(v.gate + o, s.gate + g * C, sizeof(int16_t) * C);
                        }
                        memcpy(v.pacc + (size_t)b * O, s.pacc, sizeof(int32_t) * O);
                        memcpy(v.c + (size_t)b * C, cl + (size_t)b * C, sizeof(int16_t) * C);
                        memcpy(v.m + (size_t)b * C, s.m, C);
                        memcpy(v.h + (size_t)b * O, hl + (size_t)b * O, O);
                    }
                }
            }
            free(s.acc); free(s.pacc); free(s.xg); free(s.pre); free(s.ain); free(s.gate); free(s.m);
        }

        if (tr) tr += (size_t)T * rec;
        h_off += (size_t)B * O;
        c_off += (size_t)B * C;
        in = out;
    }
    free(seq[0]); free(seq[1]);
    return 0;
}

int qref_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
