// Post-training calibration (Section 4) and the quantization recipe of Table 2 on the device.
//
// Calibration is a float (fp64) forward pass of Eq. 1-7 with a range logger on every tensor whose scale is measured;
// it runs once per model, so the kernels are plain - one thread per output - and the only care taken is that the
// logging costs no extra pass: every kernel reduces the values it produces (block-wide, then one atomic per block on an
// order-preserving integer encoding of the double).
// The quantizer's device work is what touches whole tensors: max |.| reductions and the rounding of weights and
// biases; the scalar arithmetic of Table 2 stays on the host.
#include <cuda_runtime.h>

#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/qlstm_calib.h"

namespace {

enum { ST_XMIN, ST_XMAX, ST_HMIN, ST_HMAX, ST_MMIN, ST_MMAX, ST_CABS, ST_G0, ST_COUNT = ST_G0 + 4 };

// doubles as unsigned integers with the same order
__host__ __device__ inline unsigned long long enc(double d)
{
    unsigned long long u;
    memcpy(&u, &d, 8);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}
inline double dec(unsigned long long u)
{
    u = (u >> 63) ? (u & 0x7fffffffffffffffull) : ~u;
    double d;
    memcpy(&d, &u, 8);
    return d;
}

// block-wide min / max of one value per thread into two slots (either may be null)
__device__ void log_range(double v, bool valid, unsigned long long *slot_min, unsigned long long *slot_max)
{
    unsigned long long lo = valid ? enc(v) : ~0ull, hi = valid ? enc(v) : 0ull;
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long l2 = __shfl_down_sync(0xffffffffu, lo, o), h2 = __shfl_down_sync(0xffffffffu, hi, o);
        lo = l2 < lo ? l2 : lo;
        hi = h2 > hi ? h2 : hi;
    }
    __shared__ unsigned long long s_lo[32], s_hi[32];
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    if (l == 0) { s_lo[w] = lo; s_hi[w] = hi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < (int)(blockDim.x + 31) / 32; ++i) {
            lo = s_lo[i] < lo ? s_lo[i] : lo;
            hi = s_hi[i] > hi ? s_hi[i] : hi;
        }
        if (slot_min) atomicMin(slot_min, lo);
        if (slot_max) atomicMax(slot_max, hi);
    }
    __syncthreads();
}

struct FlLayer {
    int I, C, O;
    uint32_t flags;
    const double *W[4], *R[4], *P[4], *L[4], *b[4], *Wp, *bp;     // device
};

__global__ void k_range(const double *v, size_t n, unsigned long long *slot_min, unsigned long long *slot_max)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    log_range(i < n ? v[i] : 0.0, i < n, slot_min, slot_max);
}

// gate sums a[g][b][u] = W_g x + R_g h (+ P_g c^{t-1} for i and f); the output gate's peephole waits for c^t (Eq. 5)
__global__ void k_fl_gates(FlLayer L, const double *x, const double *h, const double *c, int B, double *a)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t per = (size_t)B * L.C;
    if (i >= 4 * per) return;
    const int g = (int)(i / per);
    const int b = (int)((i - g * per) / L.C), u = (int)(i % L.C);
    if (!L.W[g]) { a[i] = 0.0; return; }
    const double *w = L.W[g] + (size_t)u * L.I, *r = L.R[g] + (size_t)u * L.O;
    const double *xb = x + (size_t)b * L.I, *hb = h + (size_t)b * L.O;
    double s = 0.0;
    for (int j = 0; j < L.I; ++j) s += w[j] * xb[j];
    double s2 = 0.0;
    for (int k = 0; k < L.O; ++k) s2 += r[k] * hb[k];
    s += s2;
    if ((L.flags & QLSTM_PEEPHOLE) && (g == 0 || g == 1)) s += L.P[g][u] * c[(size_t)b * L.C + u];
    a[i] = s;
}

// per (gate in mask, row): mean and population standard deviation of the gate sums (1 where it is 0), and max |.|
__global__ void k_fl_rowstats(FlLayer L, const double *a, int B, unsigned mask, double *mean, double *stdv, unsigned long long *stats)
{
    const int g = blockIdx.x / B, b = blockIdx.x % B;
    if (!((mask >> g) & 1u) || !L.W[g]) return;
    const double *row = a + ((size_t)g * B + b) * L.C;
    double s = 0.0, q = 0.0, m = 0.0;
    for (int u = threadIdx.x; u < L.C; u += blockDim.x) { const double v = row[u]; s += v; q += v * v; m = fmax(m, fabs(v)); }
    __shared__ double sh[3][32];
    for (int o = 16; o > 0; o >>= 1) {
        s += __shfl_down_sync(0xffffffffu, s, o);
        q += __shfl_down_sync(0xffffffffu, q, o);
        m = fmax(m, __shfl_down_sync(0xffffffffu, m, o));
    }
    if ((threadIdx.x & 31) == 0) { sh[0][threadIdx.x >> 5] = s; sh[1][threadIdx.x >> 5] = q; sh[2][threadIdx.x >> 5] = m; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < (int)blockDim.x / 32; ++i) { s += sh[0][i]; q += sh[1][i]; m = fmax(m, sh[2][i]); }
        const double mu = s / L.C;
        double var = q / L.C - mu * mu;
        double sd = sqrt(var > 0.0 ? var : 0.0);
        mean[g * B + b] = mu;
        stdv[g * B + b] = sd == 0.0 ? 1.0 : sd;
        atomicMax(stats + ST_G0 + g, enc(m));
    }
}

__device__ inline double gate_value(const FlLayer &L, const double *a, const double *mean, const double *stdv, int g, int B, int b, int u)
{
    double v = a[((size_t)g * B + b) * L.C + u];
    if (L.flags & QLSTM_LAYERNORM) v = (v - mean[g * B + b]) / stdv[g * B + b] * L.L[g][u];
    return v + L.b[g][u];
}
__device__ inline double sigm(double v) { return 1.0 / (1.0 + exp(-v)); }

// f, i, z -> c^t; the output gate's sum gets its peephole term on c^t
__global__ void k_fl_cell(FlLayer L, double *a, const double *mean, const double *stdv, double *c, int B, unsigned long long *stats)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool valid = i < (size_t)B * L.C;
    double c_new = 0.0;
    if (valid) {
        const int b = (int)(i / L.C), u = (int)(i % L.C);
        const double f = sigm(gate_value(L, a, mean, stdv, 1, B, b, u));
        const double ig = (L.flags & QLSTM_CIFG) ? 1.0 - f : sigm(gate_value(L, a, mean, stdv, 0, B, b, u));
        const double z = tanh(gate_value(L, a, mean, stdv, 2, B, b, u));
        c_new = ig * z + f * c[i];
        c[i] = c_new;
        if (L.flags & QLSTM_PEEPHOLE) a[((size_t)3 * B + b) * L.C + u] += L.P[3][u] * c_new;
    }
    log_range(fabs(c_new), valid, nullptr, stats + ST_CABS);
}

// o -> m = o tanh(c^t); without projection m is the layer output
__global__ void k_fl_out(FlLayer L, const double *a, const double *mean, const double *stdv, const double *c, int B, double *m,
                         unsigned long long *stats)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool valid = i < (size_t)B * L.C;
    double v = 0.0;
    if (valid) {
        const int b = (int)(i / L.C), u = (int)(i % L.C);
        v = sigm(gate_value(L, a, mean, stdv, 3, B, b, u)) * tanh(c[i]);
        m[i] = v;
    }
    log_range(v, valid, stats + ST_MMIN, stats + ST_MMAX);
    if (!(L.flags & QLSTM_PROJECTION)) log_range(v, valid, stats + ST_HMIN, stats + ST_HMAX);
}

__global__ void k_fl_proj(FlLayer L, const double *m, int B, double *h, unsigned long long *stats)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool valid = i < (size_t)B * L.O;
    double v = 0.0;
    if (valid) {
        const int b = (int)(i / L.O), p = (int)(i % L.O);
        const double *w = L.Wp + (size_t)p * L.C, *mb = m + (size_t)b * L.C;
        for (int u = 0; u < L.C; ++u) v += w[u] * mb[u];
        v += L.bp[p];
        h[i] = v;
    }
    log_range(v, valid, stats + ST_HMIN, stats + ST_HMAX);
}

// ---- quantizer kernels
__global__ void k_absmax(const double *v, size_t n, unsigned long long *slot)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    log_range(i < n ? fabs(v[i]) : 0.0, i < n, nullptr, slot);
}
template <class T>
__global__ void k_quant_sym(const double *v, size_t n, double scale, double qmax, T *out)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    double q = rint(v[i] / scale);                   // to nearest, ties to even: the host recipe's rounding
    q = q > qmax ? qmax : (q < -qmax ? -qmax : q);
    out[i] = (T)q;
}

struct DevBuf {
    std::vector<void *> owned;
    ~DevBuf() { for (void *p : owned) cudaFree(p); }
    template <class T> T *alloc(size_t n)
    {
        void *d = nullptr;
        if (cudaMalloc(&d, (n ? n : 1) * sizeof(T)) != cudaSuccess) return nullptr;
        owned.push_back(d);
        return (T *)d;
    }
    const double *upload(const double *h, size_t n)
    {
        double *d = alloc<double>(n);
        if (d && cudaMemcpy(d, h, n * sizeof(double), cudaMemcpyHostToDevice) != cudaSuccess) return nullptr;
        return d;
    }
};

int check_float_layer(const qlstm_float_layer_t &l)
{
    const bool proj = l.flags & QLSTM_PROJECTION, peep = l.flags & QLSTM_PEEPHOLE, ln = l.flags & QLSTM_LAYERNORM,
               cifg = l.flags & QLSTM_CIFG;
    if (l.flags & ~15u) return QLSTM_ERR_ARG;
    if (l.n_input <= 0 || l.n_cell <= 0 || l.n_output <= 0) return QLSTM_ERR_DIM;
    if (!proj && l.n_output != l.n_cell) return QLSTM_ERR_DIM;
    for (int g = 0; g < 4; ++g) {
        const bool active = !(cifg && g == 0);
        if (active && (!l.W[g] || !l.R[g] || !l.b[g] || (ln && !l.L[g]) || (peep && g != 2 && !l.P[g]))) return QLSTM_ERR_ARG;
        if (!active && (l.W[g] || l.R[g] || l.b[g])) return QLSTM_ERR_ARG;
    }
    if (proj && (!l.W_proj || !l.b_proj)) return QLSTM_ERR_ARG;
    return QLSTM_OK;
}

bool upload_layer(DevBuf &buf, const qlstm_float_layer_t &l, FlLayer &d)
{
    memset(&d, 0, sizeof(d));
    d.I = l.n_input; d.C = l.n_cell; d.O = l.n_output; d.flags = l.flags;
    for (int g = 0; g < 4; ++g) {
        if (!l.W[g]) continue;
        d.W[g] = buf.upload(l.W[g], (size_t)l.n_cell * l.n_input);
        d.R[g] = buf.upload(l.R[g], (size_t)l.n_cell * l.n_output);
        d.b[g] = buf.upload(l.b[g], l.n_cell);
        if (!d.W[g] || !d.R[g] || !d.b[g]) return false;
        if ((l.flags & QLSTM_LAYERNORM) && !(d.L[g] = buf.upload(l.L[g], l.n_cell))) return false;
        if ((l.flags & QLSTM_PEEPHOLE) && g != 2 && !(d.P[g] = buf.upload(l.P[g], l.n_cell))) return false;
    }
    if (l.flags & QLSTM_PROJECTION) {
        d.Wp = buf.upload(l.W_proj, (size_t)l.n_output * l.n_cell);
        d.bp = buf.upload(l.b_proj, l.n_output);
        if (!d.Wp || !d.bp) return false;
    }
    return true;
}

inline unsigned blocks(size_t n, int tpb) { return (unsigned)((n + tpb - 1) / tpb); }

}  // namespace

extern "C" int qlstm_calibrate(const qlstm_float_layer_t *layers, int n_layers, const double *x_host, int T, int B, int device,
                               qlstm_ranges_t *ranges_out)
{
    if (!layers || n_layers <= 0 || !x_host || T <= 0 || B <= 0 || !ranges_out) return QLSTM_ERR_ARG;
    for (int l = 0; l < n_layers; ++l) {
        int rc = check_float_layer(layers[l]);
        if (rc != QLSTM_OK) return rc;
        if (l > 0 && layers[l].n_input != layers[l - 1].n_output) return QLSTM_ERR_ARG;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return QLSTM_ERR_CUDA;
    if (cudaSetDevice(device) != cudaSuccess) return QLSTM_ERR_CUDA;
    DevBuf buf;
    const int TPB = 128;
    size_t max_o = 0;
    for (int l = 0; l < n_layers; ++l) max_o = std::max(max_o, (size_t)layers[l].n_output);
    // the sequences between layers ping-pong in two buffers
    double *seq[2] = {buf.alloc<double>((size_t)T * B * max_o), buf.alloc<double>((size_t)T * B * max_o)};
    const double *x_dev = buf.upload(x_host, (size_t)T * B * layers[0].n_input);
    unsigned long long *stats = buf.alloc<unsigned long long>((size_t)n_layers * ST_COUNT);
    if (!seq[0] || !seq[1] || !x_dev || !stats) return QLSTM_ERR_NOMEM;
    std::vector<unsigned long long> init((size_t)n_layers * ST_COUNT);
    for (int l = 0; l < n_layers; ++l) {
        unsigned long long *s = &init[(size_t)l * ST_COUNT];
        s[ST_XMIN] = s[ST_HMIN] = s[ST_MMIN] = ~0ull;
        s[ST_XMAX] = s[ST_HMAX] = s[ST_MMAX] = 0ull;
        s[ST_CABS] = enc(0.0);
        for (int g = 0; g < 4; ++g) s[ST_G0 + g] = enc(0.0);
    }
    if (cudaMemcpy(stats, init.data(), init.size() * 8, cudaMemcpyHostToDevice) != cudaSuccess) return QLSTM_ERR_CUDA;

    const double *in = x_dev;
    for (int l = 0; l < n_layers; ++l) {
        const qlstm_float_layer_t &fl = layers[l];
        FlLayer L;
        DevBuf lbuf;
        if (!upload_layer(lbuf, fl, L)) return QLSTM_ERR_NOMEM;
        const size_t bc = (size_t)B * L.C, bo = (size_t)B * L.O;
        double *a = lbuf.alloc<double>(4 * bc), *c = lbuf.alloc<double>(bc), *m = lbuf.alloc<double>(bc), *h0 = lbuf.alloc<double>(bo);
        double *mean = lbuf.alloc<double>(4 * (size_t)B), *stdv = lbuf.alloc<double>(4 * (size_t)B);
        if (!a || !c || !m || !h0 || !mean || !stdv) return QLSTM_ERR_NOMEM;
        cudaMemset(c, 0, bc * sizeof(double));
        cudaMemset(h0, 0, bo * sizeof(double));
        unsigned long long *st = stats + (size_t)l * ST_COUNT;
        double *out = seq[l & 1];
        const bool ln = fl.flags & QLSTM_LAYERNORM, proj = fl.flags & QLSTM_PROJECTION;
        k_range<<<blocks((size_t)T * B * L.I, 256), 256>>>(in, (size_t)T * B * L.I, st + ST_XMIN, st + ST_XMAX);
        for (int t = 0; t < T; ++t) {
            const double *h_prev = t ? out + (size_t)(t - 1) * bo : h0;
            double *h_t = out + (size_t)t * bo;
            k_fl_gates<<<blocks(4 * bc, TPB), TPB>>>(L, in + (size_t)t * B * L.I, h_prev, c, B, a);
            if (ln) k_fl_rowstats<<<4 * B, 256>>>(L, a, B, 0x7u, mean, stdv, st);
            k_fl_cell<<<blocks(bc, TPB), TPB>>>(L, a, mean, stdv, c, B, st);
            if (ln) k_fl_rowstats<<<4 * B, 256>>>(L, a, B, 0x8u, mean, stdv, st);
            k_fl_out<<<blocks(bc, TPB), TPB>>>(L, a, mean, stdv, c, B, proj ? m : h_t, st);
            if (proj) k_fl_proj<<<blocks(bo, TPB), TPB>>>(L, m, B, h_t, st);
        }
        if (cudaDeviceSynchronize() != cudaSuccess) return QLSTM_ERR_CUDA;
        in = out;
    }
    std::vector<unsigned long long> got((size_t)n_layers * ST_COUNT);
    if (cudaMemcpy(got.data(), stats, got.size() * 8, cudaMemcpyDeviceToHost) != cudaSuccess) return QLSTM_ERR_CUDA;
    for (int l = 0; l < n_layers; ++l) {
        const unsigned long long *s = &got[(size_t)l * ST_COUNT];
        qlstm_ranges_t &r = ranges_out[l];
        r.x_min = dec(s[ST_XMIN]); r.x_max = dec(s[ST_XMAX]);
        r.h_min = std::fmin(dec(s[ST_HMIN]), 0.0); r.h_max = std::fmax(dec(s[ST_HMAX]), 0.0);     // the initial state 0 belongs to the range
        r.m_min = dec(s[ST_MMIN]); r.m_max = dec(s[ST_MMAX]);
        r.c_absmax = dec(s[ST_CABS]);
        for (int g = 0; g < 4; ++g) r.g_absmax[g] = dec(s[ST_G0 + g]);
    }
    return QLSTM_OK;
}

// -------------------------------------------------------------------------------------------------- Table 2

struct qlstm_quantized {
    std::vector<qlstm_layer_t> layers;
    std::vector<std::vector<int8_t>> i8;
    std::vector<std::vector<int16_t>> i16;
    std::vector<std::vector<int32_t>> i32;
    std::vector<double> scales;            // per layer: s_x, s_h, s_m, s_c
};

namespace {

qlstm_scale_t encode_scale(double real)
{
    qlstm_scale_t s = {0, 0};
    if (real == 0.0) return s;
    int e = 0;
    const double frac = frexp(real, &e);                  // real = frac * 2^e, frac in [0.5, 1)
    long long m = (long long)nearbyint(frac * 2147483648.0);
    if (m == (1ll << 31)) { m /= 2; ++e; }
    s.multiplier = (int32_t)m;
    s.shift = e;
    return s;
}

void asym_params(double lo, double hi, double *scale, int *zp)
{
    lo = std::fmin(lo, 0.0);
    hi = std::fmax(hi, 0.0);
    if (hi == lo) hi = lo + 1.0;
    *scale = (hi - lo) / 255.0;
    const double z = nearbyint(-128.0 - lo / *scale);
    *zp = (int)(z < -128.0 ? -128.0 : (z > 127.0 ? 127.0 : z));
}

struct Quantizer {
    DevBuf buf;
    unsigned long long *slot = nullptr;
    bool init() { return (slot = buf.alloc<unsigned long long>(1)) != nullptr; }
    // max |v| of a host tensor, reduced on the device; the device copy stays for the rounding kernel
    bool absmax(const double *h, size_t n, const double **dev, double *out)
    {
        *dev = buf.upload(h, n);
        if (!*dev) return false;
        const unsigned long long z = enc(0.0);
        cudaMemcpy(slot, &z, 8, cudaMemcpyHostToDevice);
        k_absmax<<<blocks(n, 256), 256>>>(*dev, n, slot);
        unsigned long long u = 0;
        if (cudaMemcpy(&u, slot, 8, cudaMemcpyDeviceToHost) != cudaSuccess) return false;
        *out = dec(u);
        return true;
    }
    template <class T>
    bool round_to(const double *dev, size_t n, double scale, double qmax, std::vector<T> &out)
    {
        T *d = buf.alloc<T>(n);
        if (!d) return false;
        k_quant_sym<T><<<blocks(n, 256), 256>>>(dev, n, scale, qmax, d);
        out.resize(n);
        return cudaMemcpy(out.data(), d, n * sizeof(T), cudaMemcpyDeviceToHost) == cudaSuccess;
    }
};

double sym_scale_of(double absmax, double qmax) { return (absmax > 0.0 ? absmax : 1.0) / qmax; }

}  // namespace

extern "C" {

int qlstm_quantize_model(const qlstm_float_layer_t *layers, const qlstm_ranges_t *ranges, int n_layers, int device,
                         qlstm_quantized_t **out)
{
    if (!out) return QLSTM_ERR_ARG;
    *out = nullptr;
    if (!layers || !ranges || n_layers <= 0) return QLSTM_ERR_ARG;
    for (int l = 0; l < n_layers; ++l) {
        int rc = check_float_layer(layers[l]);
        if (rc != QLSTM_OK) return rc;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return QLSTM_ERR_CUDA;
    if (cudaSetDevice(device) != cudaSuccess) return QLSTM_ERR_CUDA;
    qlstm_quantized *q = new (std::nothrow) qlstm_quantized();
    if (!q) return QLSTM_ERR_NOMEM;
    q->layers.resize(n_layers);
    // reserve so that the vectors of vectors never move (the layer structs point into them)
    q->i8.reserve((size_t)n_layers * 9); q->i16.reserve((size_t)n_layers * 8); q->i32.reserve((size_t)n_layers * 5);
    double s_x; int zp_x;
    asym_params(ranges[0].x_min, ranges[0].x_max, &s_x, &zp_x);
    int rc = QLSTM_OK;
    for (int l = 0; l < n_layers && rc == QLSTM_OK; ++l) {
        const qlstm_float_layer_t &fl = layers[l];
        const qlstm_ranges_t &st = ranges[l];
        const bool proj = fl.flags & QLSTM_PROJECTION, peep = fl.flags & QLSTM_PEEPHOLE, ln = fl.flags & QLSTM_LAYERNORM;
        Quantizer Q;
        if (!Q.init()) { rc = QLSTM_ERR_NOMEM; break; }
        qlstm_layer_t &d = q->layers[l];
        memset(&d, 0, sizeof(d));
        double s_h, s_m; int zp_h, zp_m;
        asym_params(st.h_min, st.h_max, &s_h, &zp_h);
        if (proj) asym_params(st.m_min, st.m_max, &s_m, &zp_m); else { s_m = s_h; zp_m = zp_h; }
        int m_bits = 0;
        while ((double)(1 << m_bits) < st.c_absmax) ++m_bits;             // smallest m with 2^m >= max |c| (Section 3.2.2)
        const double s_c = ldexp(1.0, m_bits - 15);
        d.n_input = fl.n_input; d.n_cell = fl.n_cell; d.n_output = fl.n_output; d.flags = fl.flags;
        d.cell_int_bits = m_bits; d.zp_x = zp_x; d.zp_m = zp_m; d.zp_h = zp_h;
        const size_t nW = (size_t)fl.n_cell * fl.n_input, nR = (size_t)fl.n_cell * fl.n_output, nC = fl.n_cell;
        for (int g = 0; g < 4 && rc == QLSTM_OK; ++g) {
            if (!fl.W[g]) continue;
            const double *dW, *dR, *dB, *dL = nullptr, *dP = nullptr;
            double aW, aR, aB, aL = 0.0, aP = 0.0;
            if (!Q.absmax(fl.W[g], nW, &dW, &aW) || !Q.absmax(fl.R[g], nR, &dR, &aR) || !Q.absmax(fl.b[g], nC, &dB, &aB)) { rc = QLSTM_ERR_NOMEM; break; }
            const double s_W = sym_scale_of(aW, 127.0), s_R = sym_scale_of(aR, 127.0);
            q->i8.emplace_back(); q->i8.emplace_back();
            std::vector<int8_t> &Wq = q->i8[q->i8.size() - 2], &Rq = q->i8.back();
            if (!Q.round_to<int8_t>(dW, nW, s_W, 127.0, Wq) || !Q.round_to<int8_t>(dR, nR, s_R, 127.0, Rq)) { rc = QLSTM_ERR_NOMEM; break; }
            d.W[g] = Wq.data(); d.R[g] = Rq.data();
            double s_gate, s_b;
            if (ln) {
                const double gm = st.g_absmax[g];
                s_gate = (gm > 0.0 ? gm : 1.0) / 32767.0;                             // Section 3.2.5
                if (!Q.absmax(fl.L[g], nC, &dL, &aL)) { rc = QLSTM_ERR_NOMEM; break; }
                const double s_L = sym_scale_of(aL, 32767.0);
                q->i16.emplace_back();
                if (!Q.round_to<int16_t>(dL, nC, s_L, 32767.0, q->i16.back())) { rc = QLSTM_ERR_NOMEM; break; }
                d.L[g] = q->i16.back().data();
                s_b = s_L * ldexp(1.0, -10);                                          // Section 3.2.6
                d.eff_ln[g] = encode_scale(s_b / ldexp(1.0, -12));
            } else {
                s_gate = ldexp(1.0, -12);                                             // Q3.12, Section 3.2.4
                s_b = s_R * s_h;
            }
            q->i32.emplace_back();
            if (!Q.round_to<int32_t>(dB, nC, s_b, 2147483647.0, q->i32.back())) { rc = QLSTM_ERR_NOMEM; break; }
            d.b[g] = q->i32.back().data();
            d.eff_x[g] = encode_scale(s_W * s_x / s_gate);
            d.eff_h[g] = encode_scale(s_R * s_h / s_gate);
            if (peep && g != 2) {
                if (!Q.absmax(fl.P[g], nC, &dP, &aP)) { rc = QLSTM_ERR_NOMEM; break; }
                const double s_P = sym_scale_of(aP, 32767.0);
                q->i16.emplace_back();
                if (!Q.round_to<int16_t>(dP, nC, s_P, 32767.0, q->i16.back())) { rc = QLSTM_ERR_NOMEM; break; }
                d.P[g] = q->i16.back().data();
                d.eff_c[g] = encode_scale(s_P * s_c / s_gate);
            }
        }
        if (rc != QLSTM_OK) break;
        d.eff_m = encode_scale(ldexp(1.0, -30) / s_m);                                // Section 3.2.7
        if (proj) {
            const size_t nP = (size_t)fl.n_output * fl.n_cell;
            const double *dWp, *dbp;
            double aWp, abp;
            if (!Q.absmax(fl.W_proj, nP, &dWp, &aWp) || !Q.absmax(fl.b_proj, fl.n_output, &dbp, &abp)) { rc = QLSTM_ERR_NOMEM; break; }
            const double s_Wp = sym_scale_of(aWp, 127.0);
            q->i8.emplace_back();
            q->i32.emplace_back();
            if (!Q.round_to<int8_t>(dWp, nP, s_Wp, 127.0, q->i8.back()) ||
                !Q.round_to<int32_t>(dbp, fl.n_output, s_Wp * s_m, 2147483647.0, q->i32.back())) { rc = QLSTM_ERR_NOMEM; break; }
            d.W_proj = q->i8.back().data();
            d.b_proj = q->i32.back().data();
            d.eff_proj = encode_scale(s_Wp * s_m / s_h);                              // Section 3.2.8
        }
        q->scales.push_back(s_x); q->scales.push_back(s_h); q->scales.push_back(s_m); q->scales.push_back(s_c);
        s_x = s_h; zp_x = zp_h;                       // the next layer reads this layer's h
    }
    if (rc != QLSTM_OK) { delete q; return rc; }
    *out = q;
    return QLSTM_OK;
}

const qlstm_layer_t *qlstm_quantized_layers(const qlstm_quantized_t *q) { return q ? q->layers.data() : nullptr; }

int qlstm_quantized_scales(const qlstm_quantized_t *q, int layer, double *out4)
{
    if (!q || !out4 || layer < 0 || layer >= (int)q->layers.size()) return QLSTM_ERR_ARG;
    for (int i = 0; i < 4; ++i) out4[i] = q->scales[(size_t)layer * 4 + i];
    return QLSTM_OK;
}

void qlstm_quantized_destroy(qlstm_quantized_t *q) { delete q; }

}  // extern "C"
