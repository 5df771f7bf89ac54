// Host side of libqlstm.so: the C ABI declared in include/qlstm.h.
//
// qlstm_create validates the layer stack, folds the zero-point terms into int32 biases
// (Section 6 of the paper), interleaves the gate rows per cell and uploads everything once;
// qlstm_run enqueues, per layer, the batched input projection and then the recurrent part.
#include <cuda_runtime.h>

#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/qlstm.h"
#include "../../include/qlstm_debug.h"
#include "fast_kernels.h"
#include "qlstm_internal.h"

using namespace ql;

namespace {

struct LayerHost {
    LayerParams p;
    int zp_x;
    std::vector<void *> owned;      // device allocations of this layer
    FastLayer fast;                 // tensor maps and tiling of the fast kernels
};

}  // namespace

struct qlstm {
    int device = 0;
    int sm_count = 0;
    int max_T = 0, max_B = 0;
    std::vector<LayerHost> layers;
    // workspaces
    int16_t *X = nullptr;           // [max_T*max_B][max N]
    int8_t *seq[2] = {nullptr, nullptr};
    SimpleScratch scratch = {};
    FastScratch fscratch = {};
    StackSmall *stack = nullptr;    // whole-stack kernel for small batches, or null
    int *status = nullptr;          // device status word of the persistent kernel
    unsigned long long *phase_ns = nullptr;   // device phase timers of the persistent kernel (profiling)
    // staging for qlstm_run_host
    int8_t *st_x = nullptr, *st_y = nullptr, *st_h = nullptr;
    int16_t *st_c = nullptr;
    cudaStream_t own_stream = nullptr;
    cudaStream_t last_stream = nullptr;
    int impl_proj = 0, impl_rec = 0;
    // profiling
    bool profiling = false;      // level >= 1: event pairs around every launch
    bool phase_timers = false;   // level 2: device timers inside the persistent kernel
    struct Span { cudaEvent_t a, b; int kind; int launches; };
    std::vector<Span> spans;
    std::vector<cudaEvent_t> event_pool;
    qlstm_profile_t prof = {};
};

namespace {

template <class T>
cudaError_t dev_upload(LayerHost &L, const std::vector<T> &src, const T **dst)
{
    void *d = nullptr;
    size_t bytes = src.size() * sizeof(T);
    cudaError_t e = cudaMalloc(&d, bytes ? bytes : 16);
    if (e != cudaSuccess) return e;
    L.owned.push_back(d);
    if (bytes) e = cudaMemcpy(d, src.data(), bytes, cudaMemcpyHostToDevice);
    *dst = (const T *)d;
    return e;
}

bool scale_ok(const qlstm_scale_t &s)
{
    if (s.multiplier == 0) return true;
    return s.multiplier >= (1 << 30) && s.shift >= -31 && s.shift <= 30;
}

int validate_layer(const qlstm_layer_t &l)
{
    const bool proj = l.flags & QLSTM_PROJECTION, peep = l.flags & QLSTM_PEEPHOLE,
               ln = l.flags & QLSTM_LAYERNORM, cifg = l.flags & QLSTM_CIFG;
    if (l.flags & ~15u) return QLSTM_ERR_ARG;
    if (l.n_input <= 0 || l.n_cell <= 0 || l.n_output <= 0) return QLSTM_ERR_DIM;
    if (l.n_input > 32768 || l.n_cell > 32768 || l.n_output > 32768) return QLSTM_ERR_DIM;
    if (!proj && l.n_output != l.n_cell) return QLSTM_ERR_DIM;
    if (ln && l.n_cell > 8191) return QLSTM_ERR_DIM;
    if (l.cell_int_bits < 0 || l.cell_int_bits > 15) return QLSTM_ERR_ARG;
    if (l.zp_x < -128 || l.zp_x > 127 || l.zp_m < -128 || l.zp_m > 127 || l.zp_h < -128 || l.zp_h > 127)
        return QLSTM_ERR_ARG;
    if (!proj && l.zp_m != l.zp_h) return QLSTM_ERR_ARG;
    for (int g = 0; g < 4; ++g) {
        bool active = !(cifg && g == 0);
        if (active) {
            if (!l.W[g] || !l.R[g] || !l.b[g]) return QLSTM_ERR_ARG;
            if (ln && !l.L[g]) return QLSTM_ERR_ARG;
            if (peep && g != 2 && !l.P[g]) return QLSTM_ERR_ARG;
            if (!scale_ok(l.eff_x[g]) || !scale_ok(l.eff_h[g])) return QLSTM_ERR_ARG;
            if (peep && g != 2 && !scale_ok(l.eff_c[g])) return QLSTM_ERR_ARG;
            if (ln && !scale_ok(l.eff_ln[g])) return QLSTM_ERR_ARG;
        } else if (l.W[g] || l.R[g] || l.b[g] || l.P[g] || l.L[g]) {
            return QLSTM_ERR_ARG;
        }
    }
    if (!scale_ok(l.eff_m)) return QLSTM_ERR_ARG;
    if (proj && (!l.W_proj || !l.b_proj || !scale_ok(l.eff_proj))) return QLSTM_ERR_ARG;
    return QLSTM_OK;
}

// Builds the device view of one layer: interleaved rows, folded biases (Section 6).
int build_layer(const qlstm_layer_t &l, LayerHost &L)
{
    const bool proj = l.flags & QLSTM_PROJECTION, peep = l.flags & QLSTM_PEEPHOLE,
               ln = l.flags & QLSTM_LAYERNORM, cifg = l.flags & QLSTM_CIFG;
    LayerParams &p = L.p;
    memset(&p, 0, sizeof(p));
    p.I = l.n_input; p.C = l.n_cell; p.O = l.n_output;
    p.G = cifg ? 3 : 4; p.N = p.C * p.G;
    p.flags = l.flags; p.m_bits = l.cell_int_bits; p.zp_m = l.zp_m; p.zp_h = l.zp_h;
    L.zp_x = l.zp_x;
    for (int g = 0; g < 4; ++g) p.slot_of_gate[g] = -1;
    for (int gi = 0; gi < p.G; ++gi) {
        int g = cifg ? gi + 1 : gi;
        p.gate_id[gi] = g;
        p.slot_of_gate[g] = gi;
        p.eff_x[gi] = {l.eff_x[g].multiplier, l.eff_x[g].shift};
        p.eff_h[gi] = {l.eff_h[g].multiplier, l.eff_h[g].shift};
        p.eff_c[gi] = {l.eff_c[g].multiplier, l.eff_c[g].shift};
        p.eff_ln[gi] = {l.eff_ln[g].multiplier, l.eff_ln[g].shift};
    }
    p.eff_m = {l.eff_m.multiplier, l.eff_m.shift};
    p.eff_proj = {l.eff_proj.multiplier, l.eff_proj.shift};

    const size_t N = (size_t)p.N;
    std::vector<int8_t> W(N * p.I), R(N * p.O);
    std::vector<int32_t> bx(N), bh(N), bln(N, 0);
    std::vector<int16_t> P(N, 0), Lw(N, 0);
    for (int u = 0; u < p.C; ++u) {
        for (int gi = 0; gi < p.G; ++gi) {
            const int g = p.gate_id[gi];
            const size_t n = (size_t)u * p.G + gi;
            const int8_t *wrow = l.W[g] + (size_t)u * p.I, *rrow = l.R[g] + (size_t)u * p.O;
            memcpy(&W[n * p.I], wrow, p.I);
            memcpy(&R[n * p.O], rrow, p.O);
            int64_t sw = 0, sr = 0;
            for (int j = 0; j < p.I; ++j) sw += wrow[j];
            for (int k = 0; k < p.O; ++k) sr += rrow[k];
            int64_t fx = -(int64_t)l.zp_x * sw;
            int64_t fh = (ln ? 0 : (int64_t)l.b[g][u]) - (int64_t)l.zp_h * sr;
            if (fx > INT32_MAX || fx < INT32_MIN || fh > INT32_MAX || fh < INT32_MIN) return QLSTM_ERR_RANGE;
            bx[n] = (int32_t)fx;
            bh[n] = (int32_t)fh;
            if (ln) { Lw[n] = l.L[g][u]; bln[n] = l.b[g][u]; }
            if (peep && g != 2) P[n] = l.P[g][u];
        }
    }
    cudaError_t e;
    if ((e = dev_upload(L, W, &p.W)) != cudaSuccess) return QLSTM_ERR_NOMEM;
    if ((e = dev_upload(L, R, &p.R)) != cudaSuccess) return QLSTM_ERR_NOMEM;
    if ((e = dev_upload(L, bx, &p.bx)) != cudaSuccess) return QLSTM_ERR_NOMEM;
    if ((e = dev_upload(L, bh, &p.bh)) != cudaSuccess) return QLSTM_ERR_NOMEM;
    if ((e = dev_upload(L, P, &p.P)) != cudaSuccess) return QLSTM_ERR_NOMEM;
    if ((e = dev_upload(L, Lw, &p.L)) != cudaSuccess) return QLSTM_ERR_NOMEM;
    if ((e = dev_upload(L, bln, &p.bln)) != cudaSuccess) return QLSTM_ERR_NOMEM;
    if (proj) {
        std::vector<int8_t> Wp((size_t)p.O * p.C);
        std::vector<int32_t> bp(p.O);
        memcpy(Wp.data(), l.W_proj, Wp.size());
        for (int o = 0; o < p.O; ++o) {
            int64_t s = 0;
            for (int u = 0; u < p.C; ++u) s += l.W_proj[(size_t)o * p.C + u];
            int64_t f = (int64_t)l.b_proj[o] - (int64_t)l.zp_m * s;
            if (f > INT32_MAX || f < INT32_MIN) return QLSTM_ERR_RANGE;
            bp[o] = (int32_t)f;
        }
        if ((e = dev_upload(L, Wp, &p.Wproj)) != cudaSuccess) return QLSTM_ERR_NOMEM;
        if ((e = dev_upload(L, bp, &p.bp)) != cudaSuccess) return QLSTM_ERR_NOMEM;
    }
    return QLSTM_OK;
}

template <class T>
bool dmalloc(T **p, size_t count)
{
    return cudaMalloc((void **)p, (count ? count : 1) * sizeof(T)) == cudaSuccess;
}

cudaEvent_t get_event(qlstm *q)
{
    if (!q->event_pool.empty()) {
        cudaEvent_t e = q->event_pool.back();
        q->event_pool.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

struct SpanGuard {
    qlstm *q; cudaStream_t st; int kind; qlstm::Span sp; bool on;
    SpanGuard(qlstm *q_, cudaStream_t st_, int kind_) : q(q_), st(st_), kind(kind_), on(q_->profiling)
    {
        if (on) { sp.a = get_event(q); sp.b = get_event(q); sp.kind = kind; sp.launches = 0; cudaEventRecord(sp.a, st); }
    }
    void done(int launches)
    {
        if (!on) { tally(launches); return; }
        cudaEventRecord(sp.b, st);
        sp.launches = launches;
        q->spans.push_back(sp);
    }
    void tally(int launches)
    {
        if (kind == 0) q->prof.projection_launches += launches;
        else if (kind == 1) q->prof.recurrent_launches += launches;
        else q->prof.other_launches += launches;
    }
};

void collect_spans(qlstm *q)
{
    for (auto &sp : q->spans) {
        float ms = 0.f;
        cudaEventSynchronize(sp.b);
        cudaEventElapsedTime(&ms, sp.a, sp.b);
        if (sp.kind == 0) { q->prof.projection_ms += ms; q->prof.projection_launches += sp.launches; }
        else if (sp.kind == 1) { q->prof.recurrent_ms += ms; q->prof.recurrent_launches += sp.launches; }
        else { q->prof.other_ms += ms; q->prof.other_launches += sp.launches; }
        q->event_pool.push_back(sp.a);
        q->event_pool.push_back(sp.b);
    }
    q->spans.clear();
}

int run_projection(qlstm *q, LayerHost &L, const int8_t *x, int rows, int16_t *X, cudaStream_t st)
{
    SpanGuard g(q, st, 0);
    bool fast_ok = fast_projection_supported(L.fast, L.p);
    int impl = q->impl_proj;
    if (impl == 2 && !fast_ok) return QLSTM_ERR_DIM;
    bool use_fast = (impl == 2) || (impl == 0 && fast_ok);
    cudaError_t e = use_fast ? launch_projection_fast(L.fast, L.p, x, rows, X, q->sm_count, q->status, st)
                             : launch_projection_simple(L.p, x, rows, X, st);
    g.done(1);
    return e == cudaSuccess ? QLSTM_OK : QLSTM_ERR_CUDA;
}

}  // namespace

extern "C" {

int qlstm_create(const qlstm_layer_t *layers, int n_layers, int max_T, int max_B, int device, qlstm_t **out)
{
    if (!out) return QLSTM_ERR_ARG;
    *out = nullptr;
    if (!layers || n_layers <= 0 || max_T <= 0 || max_B <= 0) return QLSTM_ERR_ARG;
    for (int l = 0; l < n_layers; ++l) {
        int rc = validate_layer(layers[l]);
        if (rc != QLSTM_OK) return rc;
        if (l > 0 && (layers[l].n_input != layers[l - 1].n_output || layers[l].zp_x != layers[l - 1].zp_h))
            return QLSTM_ERR_ARG;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return QLSTM_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return QLSTM_ERR_CUDA;
    if (prop.major != 10) return QLSTM_ERR_CUDA;                 // the kernels are built for sm_100a only
    if (cudaSetDevice(device) != cudaSuccess) return QLSTM_ERR_CUDA;

    qlstm *q = new (std::nothrow) qlstm();
    if (!q) return QLSTM_ERR_NOMEM;
    q->device = device;
    q->sm_count = prop.multiProcessorCount;
    q->max_T = max_T;
    q->max_B = max_B;
    q->layers.resize(n_layers);
    int rc = QLSTM_OK;
    size_t maxN = 0, maxO = 0, maxC = 0, maxG = 4, sumO = 0, sumC = 0;
    for (int l = 0; l < n_layers && rc == QLSTM_OK; ++l) {
        rc = build_layer(layers[l], q->layers[l]);
        const LayerParams &p = q->layers[l].p;
        if ((size_t)p.N > maxN) maxN = p.N;
        if ((size_t)p.O > maxO) maxO = p.O;
        if ((size_t)p.C > maxC) maxC = p.C;
        sumO += p.O; sumC += p.C;
    }
    const size_t rows = (size_t)max_T * max_B;
    bool ok = rc == QLSTM_OK;
    if (ok) {
        ok = dmalloc(&q->X, rows * maxN) && dmalloc(&q->scratch.pre, (size_t)max_B * maxN) &&
             dmalloc(&q->scratch.po, (size_t)max_B * maxC) && dmalloc(&q->scratch.stats, (size_t)max_B * maxG * 2) &&
             dmalloc(&q->scratch.m, (size_t)max_B * maxC) && dmalloc(&q->status, 4) && dmalloc(&q->phase_ns, 8) &&
             dmalloc(&q->st_x, rows * q->layers[0].p.I) && dmalloc(&q->st_y, rows * q->layers.back().p.O) &&
             dmalloc(&q->st_h, (size_t)max_B * sumO) && dmalloc(&q->st_c, (size_t)max_B * sumC);
        if (ok && n_layers > 1) ok = dmalloc(&q->seq[0], rows * maxO) && dmalloc(&q->seq[1], rows * maxO);
        if (!ok) rc = QLSTM_ERR_NOMEM;
    }
    if (ok && cudaStreamCreateWithFlags(&q->own_stream, cudaStreamNonBlocking) != cudaSuccess) { ok = false; rc = QLSTM_ERR_CUDA; }
    if (ok) {
        cudaMemset(q->status, 0, 4 * sizeof(int));
        cudaMemset(q->phase_ns, 0, 8 * sizeof(unsigned long long));
        int frc = fast_scratch_init(q->fscratch, max_B, (int)maxC, (int)maxO, (int)maxN, q->sm_count);
        if (frc != QLSTM_OK) { ok = false; rc = frc; }
    }
    for (int l = 0; l < n_layers && ok; ++l) {
        q->layers[l].fast.proj_rows_hint = (long long)max_T * max_B;
        int frc = fast_layer_init(q->layers[l].fast, q->layers[l].p, q->fscratch, max_T, max_B);
        if (frc != QLSTM_OK) { ok = false; rc = frc; }
    }
    if (ok) {
        std::vector<const LayerParams *> lp;
        for (auto &L : q->layers) lp.push_back(&L.p);
        int src = stack_small_create(lp, max_T, max_B, q->sm_count, &q->stack);
        if (src != QLSTM_OK) { ok = false; rc = src; }
    }
    if (!ok) { qlstm_destroy(q); return rc; }
    *out = q;
    return QLSTM_OK;
}

void qlstm_destroy(qlstm_t *q)
{
    if (!q) return;
    cudaSetDevice(q->device);
    cudaDeviceSynchronize();
    for (auto &L : q->layers) {
        for (void *d : L.owned) cudaFree(d);
        fast_layer_destroy(L.fast);
    }
    fast_scratch_destroy(q->fscratch);
    stack_small_destroy(q->stack);
    cudaFree(q->X); cudaFree(q->seq[0]); cudaFree(q->seq[1]);
    cudaFree(q->scratch.pre); cudaFree(q->scratch.po); cudaFree(q->scratch.stats); cudaFree(q->scratch.m);
    cudaFree(q->status);
    cudaFree(q->phase_ns);
    cudaFree(q->st_x); cudaFree(q->st_y); cudaFree(q->st_h); cudaFree(q->st_c);
    for (auto &sp : q->spans) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
    for (auto e : q->event_pool) cudaEventDestroy(e);
    if (q->own_stream) cudaStreamDestroy(q->own_stream);
    delete q;
}

size_t qlstm_trace_bytes(const qlstm_t *q, int T, int B)
{
    if (!q || T <= 0 || B <= 0) return 0;
    size_t total = 0;
    for (auto &L : q->layers) total += (size_t)T * trace_record_bytes(B, L.p.C, L.p.O);
    return total;
}

int qlstm_run(qlstm_t *q, const int8_t *x_dev, int T, int B, int8_t *h_dev, int16_t *c_dev, int8_t *y_dev,
              void *trace_dev, void *cuda_stream)
{
    if (!q) return QLSTM_ERR_ARG;
    if (T < 0 || B < 0 || T > q->max_T || B > q->max_B) return QLSTM_ERR_ARG;
    if (T == 0 || B == 0) return QLSTM_OK;
    if (!x_dev || !h_dev || !c_dev || !y_dev) return QLSTM_ERR_ARG;
    // the kernels use 16-byte vector and bulk accesses on x, y and c (h is re-tiled and may sit anywhere)
    if ((((uintptr_t)x_dev | (uintptr_t)y_dev | (uintptr_t)c_dev) & 15) != 0) return QLSTM_ERR_ARG;
    if (trace_dev && ((uintptr_t)trace_dev & 15) != 0) return QLSTM_ERR_ARG;
    if (cudaSetDevice(q->device) != cudaSuccess) return QLSTM_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    q->last_stream = st;
    uint8_t *trace = (uint8_t *)trace_dev;
    if (trace && cudaMemsetAsync(trace, 0, qlstm_trace_bytes(q, T, B), st) != cudaSuccess) return QLSTM_ERR_CUDA;
    const int nl = (int)q->layers.size();
    // small batches: the whole stack in one launch (layers as a wavefront, input projection inside the step)
    if (!trace && (q->impl_rec == 0 || q->impl_rec >= 5) && q->impl_proj != 1) {
        if (q->impl_rec == 0 ? stack_small_preferred(q->stack, T, B) : stack_small_supported(q->stack, T, B)) {
            SpanGuard g(q, st, 1);
            const int schedule = q->impl_rec == 6 ? 1 : (q->impl_rec == 7 ? 2 : 0);
            int rc = launch_stack_small(q->stack, x_dev, T, B, h_dev, c_dev, y_dev, q->status, schedule, st);
            g.done(1);
            return rc;
        }
        if (q->impl_rec >= 5) return QLSTM_ERR_DIM;
    } else if (q->impl_rec >= 5) {
        return QLSTM_ERR_ARG;
    }
    if (cudaMemsetAsync(q->status, 0, 4 * sizeof(int), st) != cudaSuccess) return QLSTM_ERR_CUDA;
    const int8_t *in = x_dev;
    size_t h_off = 0, c_off = 0;
    for (int l = 0; l < nl; ++l) {
        LayerHost &L = q->layers[l];
        const LayerParams &p = L.p;
        int8_t *outp = (l == nl - 1) ? y_dev : q->seq[l & 1];
        int rc = run_projection(q, L, in, T * B, q->X, st);
        if (rc != QLSTM_OK) return rc;
        {
            SpanGuard g(q, st, 1);
            size_t rec = trace_record_bytes(B, p.C, p.O);
            bool fast_ok = !trace && fast_recurrent_supported(L.fast, p, B);
            int impl = q->impl_rec;
            if (impl >= 2 && !fast_ok) return trace ? QLSTM_ERR_ARG : QLSTM_ERR_DIM;
            bool use_fast = (impl >= 2) || (impl == 0 && fast_ok);
            int launches = 0;
            cudaError_t e;
            if (use_fast) {
                int frc = launch_recurrent_fast(L.fast, p, q->fscratch, q->X, T, B, h_dev + h_off, c_dev + c_off, outp,
                                                q->status, q->phase_timers ? q->phase_ns : nullptr, impl == 3 ? 0 : (impl == 4 ? 16 : 4), st,
                                                &launches);
                if (frc != QLSTM_OK) return frc;
                e = cudaSuccess;
            } else {
                e = launch_recurrent_simple(p, q->X, T, B, h_dev + h_off, c_dev + c_off, outp, q->scratch, trace, rec,
                                            st, &launches);
            }
            g.done(launches);
            if (e != cudaSuccess) return QLSTM_ERR_CUDA;
            if (trace) trace += (size_t)T * rec;
        }
        h_off += (size_t)B * p.O;
        c_off += (size_t)B * p.C;
        in = outp;
    }
    return QLSTM_OK;
}

int qlstm_run_host(qlstm_t *q, const int8_t *x_host, int T, int B, int8_t *h_host, int16_t *c_host, int8_t *y_host)
{
    if (!q) return QLSTM_ERR_ARG;
    if (T < 0 || B < 0 || T > q->max_T || B > q->max_B) return QLSTM_ERR_ARG;
    if (T == 0 || B == 0) return QLSTM_OK;
    if (!x_host || !h_host || !c_host || !y_host) return QLSTM_ERR_ARG;
    if (cudaSetDevice(q->device) != cudaSuccess) return QLSTM_ERR_CUDA;
    size_t sumO = 0, sumC = 0;
    for (auto &L : q->layers) { sumO += L.p.O; sumC += L.p.C; }
    const size_t xb = (size_t)T * B * q->layers[0].p.I, yb = (size_t)T * B * q->layers.back().p.O;
    const size_t hb = (size_t)B * sumO, cb = (size_t)B * sumC * sizeof(int16_t);
    cudaStream_t st = q->own_stream;
    if (cudaMemcpyAsync(q->st_x, x_host, xb, cudaMemcpyHostToDevice, st) != cudaSuccess) return QLSTM_ERR_CUDA;
    if (cudaMemcpyAsync(q->st_h, h_host, hb, cudaMemcpyHostToDevice, st) != cudaSuccess) return QLSTM_ERR_CUDA;
    if (cudaMemcpyAsync(q->st_c, c_host, cb, cudaMemcpyHostToDevice, st) != cudaSuccess) return QLSTM_ERR_CUDA;
    int rc = qlstm_run(q, q->st_x, T, B, q->st_h, q->st_c, q->st_y, nullptr, st);
    if (rc != QLSTM_OK) return rc;
    if (cudaMemcpyAsync(y_host, q->st_y, yb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return QLSTM_ERR_CUDA;
    if (cudaMemcpyAsync(h_host, q->st_h, hb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return QLSTM_ERR_CUDA;
    if (cudaMemcpyAsync(c_host, q->st_c, cb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return QLSTM_ERR_CUDA;
    return qlstm_last_status(q);
}

int qlstm_input_projection(qlstm_t *q, int layer, const int8_t *x_dev, int rows, int16_t *out_dev, void *cuda_stream)
{
    if (!q || layer < 0 || layer >= (int)q->layers.size() || rows < 0) return QLSTM_ERR_ARG;
    if ((size_t)rows > (size_t)q->max_T * q->max_B) return QLSTM_ERR_ARG;
    if (rows == 0) return QLSTM_OK;
    if (!x_dev || !out_dev) return QLSTM_ERR_ARG;
    if (((uintptr_t)x_dev & 15) != 0 || ((uintptr_t)out_dev & 31) != 0) return QLSTM_ERR_ARG;   // 32-byte stores to out
    if (cudaSetDevice(q->device) != cudaSuccess) return QLSTM_ERR_CUDA;
    q->last_stream = (cudaStream_t)cuda_stream;
    return run_projection(q, q->layers[layer], x_dev, rows, out_dev, (cudaStream_t)cuda_stream);
}

int qlstm_debug_ring_plan(int stages, int n_owners, int contiguous, int chunks_per_tile, int chunks_total, int *out14)
{
    return debug_ring_plan(stages, n_owners, contiguous, chunks_per_tile, chunks_total, out14);
}

int qlstm_debug_projection_plan(long long max_rows, long long rows, int n_gate_rows, int n_input, int sm_count,
                                int smem_bytes, int *out5)
{
    return debug_projection_plan(max_rows, rows, n_gate_rows, n_input, sm_count, smem_bytes, out5);
}

int qlstm_last_status(qlstm_t *q)
{
    if (!q) return QLSTM_ERR_ARG;
    if (cudaSetDevice(q->device) != cudaSuccess) return QLSTM_ERR_CUDA;
    cudaError_t e = cudaStreamSynchronize(q->last_stream);
    if (e != cudaSuccess) return QLSTM_ERR_CUDA;
    int st[4] = {0, 0, 0, 0};
    if (cudaMemcpy(st, q->status, sizeof(st), cudaMemcpyDeviceToHost) != cudaSuccess) return QLSTM_ERR_CUDA;
    return st[0] == 0 ? QLSTM_OK : QLSTM_ERR_TIMEOUT;
}

int qlstm_set_impl(qlstm_t *q, int projection_impl, int recurrent_impl)
{
    if (!q || projection_impl < 0 || projection_impl > 2 || recurrent_impl < 0 || recurrent_impl > 7) return QLSTM_ERR_ARG;
    q->impl_proj = projection_impl;
    q->impl_rec = recurrent_impl;
    return QLSTM_OK;
}

int qlstm_debug_barrier_timeout(qlstm_t *q, int missing_arrivals, unsigned long long limit_ns)
{
    if (!q || missing_arrivals < 0 || missing_arrivals > 1024) return QLSTM_ERR_ARG;
    if (missing_arrivals > 0 && (limit_ns == 0 || limit_ns > 1000000000ull)) return QLSTM_ERR_ARG;   // at most 1 s
    for (auto &L : q->layers) {
        L.fast.dbg_barrier_extra = (unsigned)missing_arrivals;
        L.fast.dbg_spin_limit_ns = missing_arrivals > 0 ? limit_ns : 0;
    }
    stack_small_debug_timeout(q->stack, (unsigned)missing_arrivals, limit_ns);
    return QLSTM_OK;
}

int qlstm_debug_activation_tables(qlstm_t *q, int enable)
{
    if (!q || enable < 0 || enable > 2) return QLSTM_ERR_ARG;
    int n = 0;
    for (auto &L : q->layers) {
        L.fast.dbg_no_tables = enable == 0;
        L.fast.dbg_general_kernel = enable == 2;
        if (L.fast.act_tab) ++n;
    }
    return n;
}

int qlstm_set_profiling(qlstm_t *q, int level)
{
    if (!q) return QLSTM_ERR_ARG;
    q->profiling = level >= 1;
    q->phase_timers = level >= 2;
    return QLSTM_OK;
}

int qlstm_get_profile(qlstm_t *q, qlstm_profile_t *out, int reset)
{
    if (!q || !out) return QLSTM_ERR_ARG;
    if (cudaSetDevice(q->device) != cudaSuccess) return QLSTM_ERR_CUDA;
    collect_spans(q);
    unsigned long long ns[8] = {0};
    if (cudaMemcpy(ns, q->phase_ns, sizeof(ns), cudaMemcpyDeviceToHost) != cudaSuccess) return QLSTM_ERR_CUDA;
    *out = q->prof;
    out->phase_a_ms = ns[0] * 1e-6; out->wait_a_ms = ns[1] * 1e-6;
    out->phase_b_ms = ns[2] * 1e-6; out->wait_b_ms = ns[3] * 1e-6;
    out->phase_c_ms = ns[4] * 1e-6; out->wait_c_ms = ns[5] * 1e-6;
    out->matmul_a_ms = ns[6] * 1e-6;
    if (reset) {
        q->prof = qlstm_profile_t{};
        cudaMemset(q->phase_ns, 0, sizeof(ns));
    }
    return QLSTM_OK;
}

int qlstm_device_info(qlstm_t *q, int *sm_count, int *persistent_blocks)
{
    if (!q) return QLSTM_ERR_ARG;
    if (sm_count) *sm_count = q->sm_count;
    if (persistent_blocks) *persistent_blocks = q->layers.empty() ? 0 : (q->layers[0].fast.rec_ok ? q->layers[0].fast.grid : 0);
    return QLSTM_OK;
}

const char *qlstm_strerror(int code)
{
    switch (code) {
        case QLSTM_OK: return "ok";
        case QLSTM_ERR_ARG: return "invalid argument";
        case QLSTM_ERR_DIM: return "dimension outside the supported range";
        case QLSTM_ERR_RANGE: return "bias with folded zero-point term does not fit int32";
        case QLSTM_ERR_NOMEM: return "out of memory";
        case QLSTM_ERR_CUDA: return "CUDA error or no sm_100 device";
        case QLSTM_ERR_LAUNCH: return "persistent kernel cannot be co-resident";
        case QLSTM_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown error";
    }
}

}  // extern "C"
