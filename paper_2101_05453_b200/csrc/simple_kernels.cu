// Simple CUDA path of the integer LSTM: one thread per output element, one launch per phase.
//
// It exists for three reasons: it is the path that writes the per-step trace, it covers every
// shape the tensor-core kernels do not (odd widths), and it cross-checks the fast kernels on
// the GPU itself.  Same arithmetic (qmath.cuh) and same packed weights as the fast path.
#include "qlstm_internal.h"

namespace ql {

__device__ __forceinline__ int32_t dot_i8(const int8_t *__restrict__ w, const int8_t *__restrict__ a, int n)
{
    int32_t acc = 0;
    int k = 0;
    if ((((uintptr_t)w | (uintptr_t)a) & 3) == 0) {
        const int32_t *w4 = (const int32_t *)w, *a4 = (const int32_t *)a;
        for (; k + 4 <= n; k += 4) acc = __dp4a(w4[k >> 2], a4[k >> 2], acc);
    }
    for (; k < n; ++k) acc += (int32_t)w[k] * (int32_t)a[k];
    return acc;
}

// Input projection (Section 3.2.4, first rescale term), all rows at once:
//   X[r][n] = sat16(rescale(sum_j W[n][j] x[r][j] + bx[n], eff_x))
__global__ void k_projection_simple(LayerParams p, const int8_t *__restrict__ x, int rows, int16_t *__restrict__ X)
{
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)rows * p.N) return;
    int n = (int)(idx % p.N);
    size_t r = idx / p.N;
    int32_t acc = dot_i8(p.W + (size_t)n * p.I, x + r * p.I, p.I) + p.bx[n];   // cannot overflow: |.| < 2^30
    X[idx] = (int16_t)sat16(mbqm(acc, p.eff_x[n % p.G]));
}

// Gate sums (Section 3.2.4 / 3.2.5): recurrent matmul + folded bias, rescale, peephole on c^{t-1}, add.
// The output gate's peephole sees c^t (Eq. 5), so with a peephole its sum is finished in k_cell.
__global__ void k_gate_pre(LayerParams p, const int16_t *__restrict__ Xt, int B, const int8_t *__restrict__ h,
                           const int16_t *__restrict__ c, SimpleScratch s, TraceRec tr)
{
    int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= B * p.N) return;
    int n = idx % p.N, b = idx / p.N;
    int u = n / p.G, gi = n % p.G, g = p.gate_id[gi];
    int32_t acc = sat32((int64_t)dot_i8(p.R + (size_t)n * p.O, h + (size_t)b * p.O, p.O) + p.bh[n]);
    int32_t H = sat16(mbqm(acc, p.eff_h[gi]));
    int32_t X = Xt[(size_t)b * p.N + n];
    bool peep = (p.flags & F_PEEPHOLE) != 0;
    if (tr.acc) {
        size_t o = ((size_t)g * B + b) * p.C + u;
        tr.acc[o] = acc;
        tr.xg[o] = (int16_t)X;
    }
    if (peep && g == 3) {
        s.po[(size_t)b * p.C + u] = X + H;
        return;
    }
    int32_t Pc = 0;
    if (peep && g != 2) Pc = sat16(mbqm((int32_t)p.P[n] * (int32_t)c[(size_t)b * p.C + u], p.eff_c[gi]));
    int32_t pre = sat16(X + H + Pc);
    s.pre[(size_t)b * p.N + n] = (int16_t)pre;
    if (tr.pre) tr.pre[((size_t)g * B + b) * p.C + u] = (int16_t)pre;
}

// Layer-norm statistics for the gates in gate_mask: one block per (row, gate slot).
__global__ void k_ln_stats(LayerParams p, int B, SimpleScratch s, unsigned gate_mask)
{
    int b = blockIdx.x / p.G, gi = blockIdx.x % p.G;
    if (!((gate_mask >> p.gate_id[gi]) & 1)) return;
    __shared__ long long sh_sum[32], sh_sq[32];
    long long sum = 0, sq = 0;
    for (int u = threadIdx.x; u < p.C; u += blockDim.x) {
        long long v = s.pre[(size_t)b * p.N + (size_t)u * p.G + gi];
        sum += v;
        sq += v * v;
    }
    for (int o = 16; o > 0; o >>= 1) {
        sum += __shfl_down_sync(0xffffffffu, sum, o);
        sq += __shfl_down_sync(0xffffffffu, sq, o);
    }
    int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    if (l == 0) { sh_sum[w] = sum; sh_sq[w] = sq; }
    __syncthreads();
    if (threadIdx.x == 0) {
        long long S = 0, Q = 0;
        for (int i = 0; i < (blockDim.x + 31) / 32; ++i) { S += sh_sum[i]; Q += sh_sq[i]; }
        LnStats st = ln_stats(S, Q, p.C);
        s.stats[((size_t)b * p.G + gi) * 2 + 0] = st.mean;
        s.stats[((size_t)b * p.G + gi) * 2 + 1] = st.sigma;
    }
}

__device__ __forceinline__ int32_t gate_input(const LayerParams &p, const SimpleScratch &s, int b, int u, int gi,
                                              int32_t pre)
{
    if (!(p.flags & F_LAYERNORM)) return pre;
    int n = u * p.G + gi;
    LnStats st;
    st.mean = s.stats[((size_t)b * p.G + gi) * 2 + 0];
    st.sigma = s.stats[((size_t)b * p.G + gi) * 2 + 1];
    return ln_apply_fast(pre, make_ln_row(st), p.L[n], p.bln[n], p.eff_ln[gi], make_fast_scale(p.eff_ln[gi]));
}

// Everything after the gate sums for one (row, cell).  `finish_o` says whether the output gate can be
// finished in this launch (false only with layer norm + peephole, where its statistics need c^t first).
__global__ void k_cell(LayerParams p, int B, int16_t *__restrict__ c, int8_t *__restrict__ h_out,
                       int8_t *__restrict__ y_t, SimpleScratch s, TraceRec tr, int finish_o)
{
    int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= B * p.C) return;
    int u = idx % p.C, b = idx / p.C;
    const bool peep = (p.flags & F_PEEPHOLE) != 0, cifg = (p.flags & F_CIFG) != 0, proj = (p.flags & F_PROJECTION) != 0;
    const int16_t *pre = s.pre + (size_t)b * p.N + (size_t)u * p.G;
    const int sf = p.slot_of_gate[1], sz = p.slot_of_gate[2], so = p.slot_of_gate[3], si = p.slot_of_gate[0];
    size_t tb = (size_t)b * p.C + u, tg = (size_t)B * p.C;

    int32_t af = gate_input(p, s, b, u, sf, pre[sf]);
    int32_t az = gate_input(p, s, b, u, sz, pre[sz]);
    int32_t f = sigmoid_q_fast(af, 3), z = tanh_q_fast(az, 3), i, ai = 0;
    if (cifg) {
        i = 32768 - f;                                       // 1 - f in Q0.15 (Section 3.2.9)
        if (i > 32767) i = 32767;
    } else {
        ai = gate_input(p, s, b, u, si, pre[si]);
        i = sigmoid_q_fast(ai, 3);
    }
    int32_t c_old = c[tb];
    int32_t c_new = cell_update_fast(i, z, f, c_old, p.m_bits);
    c[tb] = (int16_t)c_new;
    if (tr.c) {
        tr.ain[0 * tg + tb] = (int16_t)ai; tr.ain[1 * tg + tb] = (int16_t)af; tr.ain[2 * tg + tb] = (int16_t)az;
        tr.gate[0 * tg + tb] = (int16_t)i; tr.gate[1 * tg + tb] = (int16_t)f; tr.gate[2 * tg + tb] = (int16_t)z;
        tr.c[tb] = (int16_t)c_new;
        if (cifg) { tr.acc[tb] = 0; tr.xg[tb] = 0; tr.pre[tb] = 0; }
    }
    int32_t pre_o;
    if (peep) {
        int n = u * p.G + so;
        pre_o = sat16(s.po[tb] + sat16(mbqm((int32_t)p.P[n] * c_new, p.eff_c[so])));
        s.pre[(size_t)b * p.N + n] = (int16_t)pre_o;
        if (tr.pre) tr.pre[3 * tg + tb] = (int16_t)pre_o;
    } else {
        pre_o = pre[so];
    }
    if (!finish_o) return;
    int32_t ao = gate_input(p, s, b, u, so, pre_o);
    int32_t o = sigmoid_q_fast(ao, 3);
    int32_t m = hidden_q_fast(o, c_new, p.m_bits, p.eff_m, make_fast_scale(p.eff_m), p.zp_m);
    if (tr.c) { tr.ain[3 * tg + tb] = (int16_t)ao; tr.gate[3 * tg + tb] = (int16_t)o; tr.m[tb] = (int8_t)m; }
    if (proj) {
        s.m[tb] = (int8_t)m;
    } else {
        h_out[tb] = (int8_t)m;
        y_t[tb] = (int8_t)m;
        if (tr.h) { tr.h[tb] = (int8_t)m; }
    }
}

// Output gate and hidden state when layer norm and peephole are both on (second statistics pass done).
__global__ void k_out(LayerParams p, int B, const int16_t *__restrict__ c, int8_t *__restrict__ h_out,
                      int8_t *__restrict__ y_t, SimpleScratch s, TraceRec tr)
{
    int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= B * p.C) return;
    int u = idx % p.C, b = idx / p.C, so = p.slot_of_gate[3];
    size_t tb = (size_t)b * p.C + u, tg = (size_t)B * p.C;
    int32_t ao = gate_input(p, s, b, u, so, s.pre[(size_t)b * p.N + (size_t)u * p.G + so]);
    int32_t o = sigmoid_q_fast(ao, 3);
    int32_t m = hidden_q_fast(o, c[tb], p.m_bits, p.eff_m, make_fast_scale(p.eff_m), p.zp_m);
    if (tr.c) { tr.ain[3 * tg + tb] = (int16_t)ao; tr.gate[3 * tg + tb] = (int16_t)o; tr.m[tb] = (int8_t)m; }
    if (p.flags & F_PROJECTION) {
        s.m[tb] = (int8_t)m;
    } else {
        h_out[tb] = (int8_t)m;
        y_t[tb] = (int8_t)m;
        if (tr.h) tr.h[tb] = (int8_t)m;
    }
}

// Projection (Section 3.2.8): h = sat8(rescale(sat32(sum_u Wproj[p][u] m[u] + bp[p]), eff_proj) + zp_h)
__global__ void k_proj(LayerParams p, int B, int8_t *__restrict__ h_out, int8_t *__restrict__ y_t, SimpleScratch s,
                       TraceRec tr)
{
    int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= B * p.O) return;
    int o = idx % p.O, b = idx / p.O;
    int32_t acc = sat32((int64_t)dot_i8(p.Wproj + (size_t)o * p.C, s.m + (size_t)b * p.C, p.C) + p.bp[o]);
    int32_t h = sat8(mbqm(acc, p.eff_proj) + p.zp_h);
    h_out[idx] = (int8_t)h;
    y_t[idx] = (int8_t)h;
    if (tr.pacc) { tr.pacc[idx] = acc; tr.h[idx] = (int8_t)h; }
}

cudaError_t launch_projection_simple(const LayerParams &p, const int8_t *x, int rows, int16_t *X, cudaStream_t st)
{
    size_t total = (size_t)rows * p.N;
    if (total == 0) return cudaSuccess;
    unsigned blocks = (unsigned)((total + 255) / 256);
    k_projection_simple<<<blocks, 256, 0, st>>>(p, x, rows, X);
    return cudaGetLastError();
}

cudaError_t launch_recurrent_simple(const LayerParams &p, const int16_t *X, int T, int B, int8_t *h, int16_t *c,
                                    int8_t *y, const SimpleScratch &s, uint8_t *trace, size_t trace_stride,
                                    cudaStream_t st, int *launches)
{
    const bool ln = (p.flags & F_LAYERNORM) != 0, peep = (p.flags & F_PEEPHOLE) != 0, proj = (p.flags & F_PROJECTION) != 0;
    const int TPB = 128;
    int n_launch = 0;
    for (int t = 0; t < T; ++t) {
        TraceRec tr = {};
        if (trace) tr = trace_view(trace + (size_t)t * trace_stride, B, p.C, p.O);
        const int16_t *Xt = X + (size_t)t * B * p.N;
        int8_t *yt = y + (size_t)t * B * p.O;
        k_gate_pre<<<(B * p.N + TPB - 1) / TPB, TPB, 0, st>>>(p, Xt, B, h, c, s, tr);
        ++n_launch;
        if (ln) {
            unsigned mask = (peep ? 0x7u : 0xFu);
            k_ln_stats<<<B * p.G, 256, 0, st>>>(p, B, s, mask);
            ++n_launch;
        }
        int finish_o = !(ln && peep);
        k_cell<<<(B * p.C + TPB - 1) / TPB, TPB, 0, st>>>(p, B, c, h, yt, s, tr, finish_o);
        ++n_launch;
        if (!finish_o) {
            k_ln_stats<<<B * p.G, 256, 0, st>>>(p, B, s, 0x8u);
            k_out<<<(B * p.C + TPB - 1) / TPB, TPB, 0, st>>>(p, B, c, h, yt, s, tr);
            n_launch += 2;
        }
        if (proj) {
            k_proj<<<(B * p.O + TPB - 1) / TPB, TPB, 0, st>>>(p, B, h, yt, s, tr);
            ++n_launch;
        }
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (launches) *launches = n_launch;
    return cudaSuccess;
}

}  // namespace ql
