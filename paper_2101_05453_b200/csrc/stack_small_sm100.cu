// Whole-stack kernel for small batches (B <= 4): every layer and every time step in ONE cooperative launch.
//
// At batch 1..4 a layer-step is a handful of mat-vec products, far too small to fill the machine, and a stack run layer
// after layer leaves all but one layer's worth of work idle.  Here the blocks are split into one group per layer and
// the layers run as a wavefront (Section 7: stacked layers are loops over the same cell): while group l works on step
// t, group l + 1 works on step t - 1.  Nothing is hoisted out of the time loop: the input contribution W x_t of
// Section 3.2.4 is a mat-vec of the step itself, so the same kernel serves a call of one time step (streaming: the
// state h, c goes in and out through the caller's buffers, Section 3.2.2) and a call of hundreds.
//
// A block owns a range of cells of its layer (all their gate rows) and a range of projection rows.  Per step:
//   X   input term       W rows x x_t (from the layer below, or the caller's x)  -> rescaled int16
//   H   recurrent term   R rows x h^{t-1} + folded bias -> rescaled, + X (+ peephole on c^{t-1}) -> gate sums (shared memory)
//       [layer norm: the block's per-row sums go to global memory; group barrier; every block adds the group's shares]
//   E   elementwise      layer norm, integer sigmoid / tanh, CIFG, cell update (c stays in shared memory), hidden state m
//       [layer norm + peephole: second exchange for the output gate, whose sum needs c^t]
//       [projection: group barrier; W_proj rows x m^t -> h^t]
//   the block then arrives on its layer's step counter; the same counter releases the layer's next step and step t of
//   the layer above.
// Weights are streamed from L2 / HBM every step with 16-byte loads (a stack's weights do not fit in shared memory:
// 94 MB for eight 2048-cell layers), dp4a accumulates, lanes that share a row reduce with shuffles.
//
// Every wait is bounded by a time limit; on expiry the waiting block sets the abort word, all blocks see it at their
// next wait and leave, and the host reports QLSTM_ERR_TIMEOUT.
#include <cstring>
#include <vector>

#include "../../include/qlstm.h"
#include "fast_kernels.h"

namespace ql {

namespace {

constexpr int SK_THREADS = 640;
constexpr int SK_WARPS = SK_THREADS / 32;
constexpr unsigned long long SK_WAIT_LIMIT_NS = 2000000000ull;     // 2 s per wait

// counters of one layer (monotonic over a call): arrivals after the gate sums (layer norm), after the output gate's
// sums (layer norm + peephole), after the hidden state (projection), and at the end of a step
enum { CNT_A = 0, CNT_A2 = 1, CNT_M = 2, CNT_H = 3, CNT_PER_LAYER = 16 };      // 64 bytes apart

struct SkLayer {
    int I, C, O, G, N;
    uint32_t flags;
    int m_bits, zp_m, zp_h;
    const int8_t *W, *R, *Wproj;
    const int32_t *bx, *bh, *bp, *bln;
    const int16_t *P, *L;
    Scale eff_x[4], eff_h[4], eff_c[4], eff_ln[4], eff_m, eff_proj;
    int cta0, n_cta;               // the layer's group of blocks
    int cpc;                       // cells per block
    int rpc;                       // projection rows per block
    int8_t *seq;                   // [max_T][B][O] this layer's output sequence (null for the last layer: the caller's y)
    int8_t *m;                     // [B][C] hidden state before the projection
    long long *part;               // [n_cta][B][4][2] layer-norm shares of the group's blocks
    size_t h_off, c_off;           // offsets of this layer in the caller's h / c state, in units of one batch row
};

struct SkCall {
    int T, B, n_layers;
    const int8_t *x;               // [T][B][I_0]
    int8_t *h;                     // caller state, layer after layer [B][O_l]
    int16_t *c;                    // [B][C_l]
    int8_t *y;                     // [T][B][O_last]
    unsigned *cnt;                 // [n_layers][CNT_PER_LAYER] counters, zero at launch
    unsigned *abort_word;
    int *status;
    unsigned long long wait_limit_ns;
    unsigned missing_arrivals;     // 0; a test makes every counter wait for arrivals that never come
};

__device__ __forceinline__ unsigned sk_ld_acquire(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long sk_timer()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)::"memory");
    return t;
}
__device__ __forceinline__ uint4 ld_stream(const uint4 *p)         // weights: read-only, no reuse inside a step
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ int32_t sk_add_sat(int32_t a, int32_t b)
{
    int32_t d;
    asm("add.sat.s32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ int32_t sk_rescale(int32_t x, const Scale &s)
{
    return s.shift <= 0 ? fast_rescale(x, make_fast_scale(s)) : mbqm(x, s);
}

// all threads of the block: publish this block's writes and add one arrival to `cnt`
__device__ __forceinline__ void sk_arrive(unsigned *cnt)
{
    __syncthreads();
    if (threadIdx.x == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(cnt) : "memory");
}
// all threads: wait until `cnt` has reached `target` (bounded); returns false once the abort word is set
__device__ __forceinline__ bool sk_wait(const SkCall &k, const unsigned *cnt, unsigned target, int *abort_s)
{
    if (threadIdx.x == 0) {
        target += k.missing_arrivals;
        if (sk_ld_acquire(cnt) < target) {
            const unsigned long long t0 = sk_timer();
            unsigned spins = 0;
            while (sk_ld_acquire(cnt) < target) {
                if ((++spins & 31u) == 0u) {
                    if (sk_ld_acquire(k.abort_word) != 0u) { *abort_s = 1; break; }
                    if (sk_timer() - t0 > k.wait_limit_ns) {
                        atomicExch(k.abort_word, 1u);
                        *abort_s = 1;
                        break;
                    }
                }
            }
        }
    }
    __syncthreads();
    return *abort_s == 0;
}

// rows [0, nrows) of a row-major int8 matrix (K bytes per row, K a multiple of 16) times NB vectors held in shared
// memory as [NB][K]; emit(row, b, acc) runs once per (row, b < NB) on one lane.  gs lanes share a row (a power of two
// that divides the number of 16-byte chunks of a row, so that every lane takes the same number of chunks CPL).
template <int NB, int CPL, class F>
__device__ __forceinline__ void matvec_rows_t(const int8_t *rows, int nrows, int K, int gs, const int8_t *vec_s, F emit)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lg = lane & (gs - 1), sub = lane / gs, rpw = 32 / gs;
    const int chunks = K >> 4;
    const int cpl = CPL > 0 ? CPL : chunks / gs;
    for (int r0 = warp * rpw; r0 < nrows; r0 += SK_WARPS * rpw) {
        const int r = r0 + sub;
        const bool valid = r < nrows;
        int32_t acc[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) acc[b] = 0;
        if (valid) {
            const uint4 *wp = reinterpret_cast<const uint4 *>(rows + (size_t)r * K) + lg;
            if (CPL > 0) {
                uint4 w[CPL > 0 ? CPL : 1];
#pragma unroll
                for (int j = 0; j < CPL; ++j) w[j] = ld_stream(wp + j * gs);             // all loads of the row in flight
#pragma unroll
                for (int j = 0; j < CPL; ++j) {
#pragma unroll
                    for (int b = 0; b < NB; ++b) {
                        const uint4 v = reinterpret_cast<const uint4 *>(vec_s + (size_t)b * K)[lg + j * gs];
                        acc[b] = __dp4a((int)w[j].x, (int)v.x, acc[b]);
                        acc[b] = __dp4a((int)w[j].y, (int)v.y, acc[b]);
                        acc[b] = __dp4a((int)w[j].z, (int)v.z, acc[b]);
                        acc[b] = __dp4a((int)w[j].w, (int)v.w, acc[b]);
                    }
                }
            } else {
#pragma unroll 4
                for (int j = 0; j < cpl; ++j) {
                    const uint4 w = ld_stream(wp + j * gs);
#pragma unroll
                    for (int b = 0; b < NB; ++b) {
                        const uint4 v = reinterpret_cast<const uint4 *>(vec_s + (size_t)b * K)[lg + j * gs];
                        acc[b] = __dp4a((int)w.x, (int)v.x, acc[b]);
                        acc[b] = __dp4a((int)w.y, (int)v.y, acc[b]);
                        acc[b] = __dp4a((int)w.z, (int)v.z, acc[b]);
                        acc[b] = __dp4a((int)w.w, (int)v.w, acc[b]);
                    }
                }
            }
        }
        for (int off = gs >> 1; off > 0; off >>= 1) {
#pragma unroll
            for (int b = 0; b < NB; ++b) acc[b] += __shfl_xor_sync(0xffffffffu, acc[b], off);
        }
        if (valid) {
#pragma unroll
            for (int b = 0; b < NB; ++b)
                if ((b & (gs - 1)) == lg) emit(r, b, acc[b]);        // the lanes of a row share out the batch rows
        }
    }
}

// lanes per row: the largest power of two (at most 32) that divides the chunks of a row
__host__ __device__ inline int lanes_per_row(int K)
{
    const int chunks = K >> 4;
    int gs = 32;
    while (gs > 1 && chunks % gs != 0) gs >>= 1;
    return gs;
}

template <int NB, class F>
__device__ __forceinline__ void matvec_rows(const int8_t *rows, int nrows, int K, const int8_t *vec_s, F emit)
{
    const int gs = lanes_per_row(K);
    switch ((K >> 4) / gs) {
        case 1: matvec_rows_t<NB, 1>(rows, nrows, K, gs, vec_s, emit); break;
        case 2: matvec_rows_t<NB, 2>(rows, nrows, K, gs, vec_s, emit); break;
        case 4: matvec_rows_t<NB, 4>(rows, nrows, K, gs, vec_s, emit); break;
        case 5: matvec_rows_t<NB, 5>(rows, nrows, K, gs, vec_s, emit); break;
        default: matvec_rows_t<NB, 0>(rows, nrows, K, gs, vec_s, emit); break;
    }
}

// [B][K] bytes from global memory written by other blocks (L2 loads) into shared memory as [NB][K], rows >= B zero
__device__ __forceinline__ void stage_vec(int8_t *dst_s, const int8_t *src, int B, int NB, int K)
{
    const int per_row = K >> 4;
    for (int i = threadIdx.x; i < NB * per_row; i += SK_THREADS) {
        const int b = i / per_row;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (b < B) v = __ldcg(reinterpret_cast<const uint4 *>(src) + i);
        reinterpret_cast<uint4 *>(dst_s)[i] = v;
    }
}
// the same for a source with any alignment (the caller's h)
__device__ __forceinline__ void stage_vec_bytes(int8_t *dst_s, const int8_t *src, int B, int NB, int K)
{
    for (int i = threadIdx.x; i < NB * K; i += SK_THREADS) dst_s[i] = (i < B * K) ? src[i] : (int8_t)0;
}

struct SkSmem {
    int8_t *x_s, *h_s, *m_s;       // staged operands [NB][I], [NB][O], [NB][C]
    int16_t *xs_s;                 // [NB][npc] rescaled input term
    int16_t *pre_s;                // [NB][npc] gate sums
    int16_t *ho_s;                 // [NB][cpc] peephole: recurrent term of the output gate (its X stays in pre_s)
    int16_t *c_s;                  // [NB][cpc] cell state of the block's cells, resident over the call
    LnRow *ln_s;                   // [NB][4]
};

template <int NB>
__global__ void __launch_bounds__(SK_THREADS, 1) k_stack_small(const SkLayer *__restrict__ layers, SkCall k)
{
    extern __shared__ __align__(16) uint8_t sk_smem[];
    __shared__ SkLayer L;
    __shared__ int abort_s;
    const int cta = blockIdx.x;
    // which layer this block belongs to
    int li = -1;
    for (int l = 0; l < k.n_layers; ++l)
        if (cta >= layers[l].cta0 && cta < layers[l].cta0 + layers[l].n_cta) li = l;
    if (li < 0) return;                                        // spare block: takes no part in any counter
    if (threadIdx.x == 0) { L = layers[li]; abort_s = 0; }
    __syncthreads();

    const int B = k.B, T = k.T;
    const int G = L.G, I = L.I, C = L.C, O = L.O;
    const bool proj = (L.flags & F_PROJECTION) != 0, ln = (L.flags & F_LAYERNORM) != 0, peep = (L.flags & F_PEEPHOLE) != 0;
    const int SF = (G == 4) ? 1 : 0, SZ = SF + 1, SO = SF + 2;
    const int rank = cta - L.cta0;                             // block within the group
    const int u0 = rank * L.cpc;
    int cells = C - u0 < L.cpc ? C - u0 : L.cpc;
    if (cells < 0) cells = 0;
    const int npc = L.cpc * G, n0 = u0 * G, n_cnt = cells * G;
    const int p_lo = rank * L.rpc;
    int p_cnt = proj ? (O - p_lo < L.rpc ? O - p_lo : L.rpc) : 0;
    if (p_cnt < 0) p_cnt = 0;

    SkSmem s;
    {
        uint8_t *p = sk_smem;
        s.x_s = (int8_t *)p;  p += (size_t)NB * I;
        s.h_s = (int8_t *)p;  p += (size_t)NB * O;
        s.m_s = (int8_t *)p;  p += proj ? (size_t)NB * C : 0;
        s.xs_s = (int16_t *)p; p += (size_t)NB * npc * 2;
        s.pre_s = (int16_t *)p; p += (size_t)NB * npc * 2;
        s.ho_s = (int16_t *)p; p += (size_t)NB * L.cpc * 2;
        s.c_s = (int16_t *)p;  p += (size_t)NB * L.cpc * 2;
        p = (uint8_t *)(((uintptr_t)p + 15) & ~(uintptr_t)15);
        s.ln_s = (LnRow *)p;
    }
    unsigned *cnt = k.cnt + (size_t)li * CNT_PER_LAYER;
    const unsigned *cnt_below = li > 0 ? k.cnt + (size_t)(li - 1) * CNT_PER_LAYER + CNT_H : nullptr;
    const unsigned n_below = li > 0 ? (unsigned)layers[li - 1].n_cta : 0u;
    const unsigned n_grp = (unsigned)L.n_cta;
    const int8_t *in_seq = li > 0 ? layers[li - 1].seq : k.x;  // [T][B][I]
    int8_t *out_seq = L.seq ? L.seq : k.y;                     // [T][B][O]
    int8_t *h_state = k.h + L.h_off * B;
    int16_t *c_state = k.c + L.c_off * B;

    // cell state of the block's cells
    for (int i = threadIdx.x; i < B * cells; i += SK_THREADS) {
        const int b = i / cells, ul = i - b * cells;
        s.c_s[b * L.cpc + ul] = c_state[(size_t)b * C + u0 + ul];
    }
    __syncthreads();

    // ---- input term of step t: waits for x_t from the layer below
    auto input_term = [&](int t) -> bool {
        if (li > 0 && !sk_wait(k, cnt_below, (unsigned)(t + 1) * n_below, &abort_s)) return false;
        stage_vec(s.x_s, in_seq + (size_t)t * B * I, B, NB, I);
        __syncthreads();
        matvec_rows<NB>(L.W + (size_t)n0 * I, n_cnt, I, s.x_s, [&](int n, int b, int32_t acc) {
            if (b < B) s.xs_s[b * npc + n] = (int16_t)sat16(sk_rescale(acc + L.bx[n0 + n], L.eff_x[n % G]));
        });
        return true;
    };

    // layer-norm constants of the rows for the gate slots in `slots`, from the group's shares
    auto exchange_stats = [&](int round, unsigned slots, unsigned *counter, unsigned target) -> bool {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        long long *mine = L.part + ((size_t)rank * 2 + round) * B * 8;
        for (int task = warp; task < B * 4; task += SK_WARPS) {
            const int b = task >> 2, gi = task & 3;
            if (!((slots >> gi) & 1u)) continue;
            long long sum = 0, sq = 0;
            for (int ul = lane; ul < cells; ul += 32) {
                const int32_t v = s.pre_s[b * npc + ul * G + gi];
                sum += v;
                sq += (long long)(v * v);
            }
            for (int o = 16; o > 0; o >>= 1) {
                sum += __shfl_down_sync(0xffffffffu, sum, o);
                sq += __shfl_down_sync(0xffffffffu, sq, o);
            }
            if (lane == 0) { mine[task * 2] = sum; mine[task * 2 + 1] = sq; }
        }
        sk_arrive(counter);
        if (!sk_wait(k, counter, target, &abort_s)) return false;
        for (int task = warp; task < B * 4; task += SK_WARPS) {
            const int gi = task & 3;
            if (!((slots >> gi) & 1u)) continue;
            long long sum = 0, sq = 0;
            for (int r = lane; r < L.n_cta; r += 32) {
                const long long *share = L.part + ((size_t)r * 2 + round) * B * 8 + task * 2;
                sum += __ldcg(share);
                sq += __ldcg(share + 1);
            }
            for (int o = 16; o > 0; o >>= 1) {
                sum += __shfl_down_sync(0xffffffffu, sum, o);
                sq += __shfl_down_sync(0xffffffffu, sq, o);
            }
            if (lane == 0) s.ln_s[task] = make_ln_row(ln_stats(sum, sq, C));
        }
        __syncthreads();
        return true;
    };

    bool ok = input_term(0);
    for (int t = 0; t < T && ok; ++t) {
        // ---- recurrent term: h^{t-1} is the previous row block of this layer's output (the caller's h at t = 0)
        if (t == 0) {
            stage_vec_bytes(s.h_s, h_state, B, NB, O);
        } else {
            stage_vec(s.h_s, out_seq + (size_t)(t - 1) * B * O, B, NB, O);
        }
        __syncthreads();
        matvec_rows<NB>(L.R + (size_t)n0 * O, n_cnt, O, s.h_s, [&](int n, int b, int32_t acc) {
            if (b >= B) return;
            const int gi = n % G, ul = n / G;
            const int32_t H = sat16(sk_rescale(sk_add_sat(acc, L.bh[n0 + n]), L.eff_h[gi]));
            const int32_t X = s.xs_s[b * npc + n];
            if (peep && gi == SO) {
                s.pre_s[b * npc + n] = (int16_t)X;               // finished after the cell update (Eq. 5: o sees c^t)
                s.ho_s[b * L.cpc + ul] = (int16_t)H;
            } else {
                int32_t v = X + H;
                if (peep && gi != SZ) v += sat16(sk_rescale((int32_t)L.P[n0 + n] * s.c_s[b * L.cpc + ul], L.eff_c[gi]));
                s.pre_s[b * npc + n] = (int16_t)sat16(v);
            }
        });
        __syncthreads();
        if (ln) {
            const unsigned all = (1u << G) - 1u;
            ok = exchange_stats(0, peep ? (all & ~(1u << SO)) : all, cnt + CNT_A, (unsigned)(t + 1) * n_grp);
            if (!ok) break;
        }

        // ---- elementwise, one cell per thread
        for (int i = threadIdx.x; i < B * cells; i += SK_THREADS) {
            const int b = i / cells, ul = i - b * cells;
            const int nl = ul * G, n = n0 + nl;
            const int16_t *pre = s.pre_s + b * npc + nl;
            const LnRow *lr = s.ln_s + b * 4;
            // input of the nonlinearity of gate slot g: the gate sum, after layer norm when the layer has it
            auto gate_in = [&](int g) -> int32_t {
                const int32_t v = pre[g];
                return ln ? ln_apply_fast(v, lr[g], L.L[n + g], L.bln[n + g], L.eff_ln[g], make_fast_scale(L.eff_ln[g])) : v;
            };
            const int32_t f = sigmoid_q_fast(gate_in(SF), 3), z = tanh_q_fast(gate_in(SZ), 3);
            int32_t ig;
            if (G == 4) ig = sigmoid_q_fast(gate_in(0), 3);
            else { ig = 32768 - f; if (ig > 32767) ig = 32767; }    // coupled input gate, Section 3.2.9
            const int32_t c_old = s.c_s[b * L.cpc + ul];
            const int32_t c_new = cell_update_fast(ig, z, f, c_old, L.m_bits);
            s.c_s[b * L.cpc + ul] = (int16_t)c_new;
            int32_t ao = peep ? (int32_t)pre[SO] : gate_in(SO);
            if (peep) {
                ao = sat16(ao + s.ho_s[b * L.cpc + ul] + sat16(sk_rescale((int32_t)L.P[n + SO] * c_new, L.eff_c[SO])));
                if (ln) { s.pre_s[b * npc + nl + SO] = (int16_t)ao; continue; }      // waits for the row's statistics
            }
            const int32_t mq = hidden_q_fast(sigmoid_q_fast(ao, 3), c_new, L.m_bits, L.eff_m, make_fast_scale(L.eff_m), L.zp_m);
            if (proj) L.m[(size_t)b * C + u0 + ul] = (int8_t)mq;
            else out_seq[((size_t)t * B + b) * O + u0 + ul] = (int8_t)mq;
        }
        if (ln && peep) {
            __syncthreads();
            ok = exchange_stats(1, 1u << SO, cnt + CNT_A2, (unsigned)(t + 1) * n_grp);
            if (!ok) break;
            for (int i = threadIdx.x; i < B * cells; i += SK_THREADS) {
                const int b = i / cells, ul = i - b * cells;
                const int n = n0 + ul * G + SO;
                const int32_t ao = ln_apply_fast(s.pre_s[b * npc + ul * G + SO], s.ln_s[b * 4 + SO], L.L[n], L.bln[n], L.eff_ln[SO],
                                                 make_fast_scale(L.eff_ln[SO]));
                const int32_t mq = hidden_q_fast(sigmoid_q_fast(ao, 3), s.c_s[b * L.cpc + ul], L.m_bits, L.eff_m,
                                                 make_fast_scale(L.eff_m), L.zp_m);
                if (proj) L.m[(size_t)b * C + u0 + ul] = (int8_t)mq;
                else out_seq[((size_t)t * B + b) * O + u0 + ul] = (int8_t)mq;
            }
        }

        // ---- projection (Section 3.2.8): needs every m of the layer
        if (proj) {
            sk_arrive(cnt + CNT_M);
            ok = sk_wait(k, cnt + CNT_M, (unsigned)(t + 1) * n_grp, &abort_s);
            if (!ok) break;
            stage_vec(s.m_s, L.m, B, NB, C);
            __syncthreads();
            matvec_rows<NB>(L.Wproj + (size_t)p_lo * C, p_cnt, C, s.m_s, [&](int r, int b, int32_t acc) {
                if (b >= B) return;
                const int32_t hq = sat8(sk_rescale(sk_add_sat(acc, L.bp[p_lo + r]), L.eff_proj) + L.zp_h);
                out_seq[((size_t)t * B + b) * O + p_lo + r] = (int8_t)hq;
            });
        }
        // ---- end of the step: h^t is complete once every block of the group has arrived.  The input term of the next
        // step does not need it, so it runs between the arrival and the wait.
        sk_arrive(cnt + CNT_H);
        if (t + 1 < T) {
            ok = input_term(t + 1);
            if (!ok) break;
        }
        ok = sk_wait(k, cnt + CNT_H, (unsigned)(t + 1) * n_grp, &abort_s);
    }

    if (!ok) {
        if (threadIdx.x == 0) atomicExch(k.status, 2);
        return;
    }
    // ---- state back to the caller: c of the block's cells; h = the last row block of the output sequence
    for (int i = threadIdx.x; i < B * cells; i += SK_THREADS) {
        const int b = i / cells, ul = i - b * cells;
        c_state[(size_t)b * C + u0 + ul] = s.c_s[b * L.cpc + ul];
    }
    if (T > 0) {
        // every block copies the part of h that belongs to its share of the output columns
        const int per = (O + L.n_cta - 1) / L.n_cta, o_lo = rank * per;
        const int o_hi = o_lo + per < O ? o_lo + per : O;
        for (int b = 0; b < B; ++b)
            for (int o = o_lo + (int)threadIdx.x; o < o_hi; o += SK_THREADS)
                h_state[(size_t)b * O + o] = __ldcg(out_seq + ((size_t)(T - 1) * B + b) * O + o);
    }
}

size_t sk_smem_bytes(const LayerParams &p, int cpc, int NB)
{
    const bool proj = (p.flags & F_PROJECTION) != 0;
    const size_t npc = (size_t)cpc * p.G;
    return (size_t)NB * p.I + (size_t)NB * p.O + (proj ? (size_t)NB * p.C : 0) + 2 * (size_t)NB * npc * 2 + 2 * (size_t)NB * cpc * 2 + 16 +
           (size_t)NB * 4 * sizeof(LnRow) + 64;
}

}  // namespace

struct StackSmall {
    bool ok = false;
    int n_layers = 0, grid = 0, max_T = 0, max_B = 0;
    size_t smem = 0;
    SkLayer *layers_dev = nullptr;
    std::vector<SkLayer> layers;
    std::vector<void *> owned;
    unsigned *cnt = nullptr;       // counters + abort word
    size_t cnt_words = 0;
    unsigned dbg_missing = 0;
    unsigned long long dbg_limit_ns = 0;
};

static const void *sk_kernel(int NB)
{
    return NB == 1 ? (const void *)k_stack_small<1> : NB == 2 ? (const void *)k_stack_small<2> : (const void *)k_stack_small<4>;
}

void stack_small_destroy(StackSmall *s)
{
    if (!s) return;
    for (void *p : s->owned) cudaFree(p);
    delete s;
}

// Plans the whole-stack kernel for a handle; *out stays null when the stack does not qualify (the per-layer kernels
// then run).  max_B beyond STACK_SMALL_MAX_B is fine: the kernel is only used for smaller batches.
int stack_small_create(const std::vector<const LayerParams *> &lp, int max_T, int max_B, int sm_count, StackSmall **out)
{
    *out = nullptr;
    const int n = (int)lp.size();
    if (n < 1 || n > sm_count) return QLSTM_OK;
    for (const LayerParams *p : lp)
        if (p->I % 16 != 0 || p->O % 16 != 0 || p->C % 16 != 0) return QLSTM_OK;
    StackSmall *s = new StackSmall();
    s->n_layers = n;
    s->grid = sm_count;
    s->max_T = max_T;
    s->max_B = max_B < STACK_SMALL_MAX_B ? max_B : STACK_SMALL_MAX_B;
    const int per = sm_count / n;
    int dev = 0, max_smem = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    size_t h_off = 0, c_off = 0;
    bool fits = true;
    for (int l = 0; l < n; ++l) {
        const LayerParams &p = *lp[l];
        SkLayer L;
        memset(&L, 0, sizeof(L));
        L.I = p.I; L.C = p.C; L.O = p.O; L.G = p.G; L.N = p.N;
        L.flags = p.flags; L.m_bits = p.m_bits; L.zp_m = p.zp_m; L.zp_h = p.zp_h;
        L.W = p.W; L.R = p.R; L.Wproj = p.Wproj; L.bx = p.bx; L.bh = p.bh; L.bp = p.bp; L.bln = p.bln; L.P = p.P; L.L = p.L;
        for (int g = 0; g < 4; ++g) { L.eff_x[g] = p.eff_x[g]; L.eff_h[g] = p.eff_h[g]; L.eff_c[g] = p.eff_c[g]; L.eff_ln[g] = p.eff_ln[g]; }
        L.eff_m = p.eff_m; L.eff_proj = p.eff_proj;
        L.cta0 = l * per; L.n_cta = per;
        L.cpc = (p.C + per - 1) / per;
        L.rpc = (p.O + per - 1) / per;
        L.h_off = h_off; L.c_off = c_off;
        h_off += p.O; c_off += p.C;
        const size_t need = sk_smem_bytes(p, L.cpc, STACK_SMALL_MAX_B);
        if (need > (size_t)max_smem) fits = false;
        if (need > s->smem) s->smem = need;
        void *d = nullptr;
        if (l + 1 < n) {
            if (cudaMalloc(&d, (size_t)max_T * s->max_B * p.O) != cudaSuccess) { stack_small_destroy(s); return QLSTM_ERR_NOMEM; }
            s->owned.push_back(d);
            L.seq = (int8_t *)d;
        }
        if (cudaMalloc(&d, (size_t)s->max_B * p.C) != cudaSuccess) { stack_small_destroy(s); return QLSTM_ERR_NOMEM; }
        s->owned.push_back(d);
        L.m = (int8_t *)d;
        if (cudaMalloc(&d, (size_t)per * 2 * s->max_B * 8 * sizeof(long long)) != cudaSuccess) { stack_small_destroy(s); return QLSTM_ERR_NOMEM; }
        s->owned.push_back(d);
        L.part = (long long *)d;
        s->layers.push_back(L);
    }
    if (!fits) { stack_small_destroy(s); return QLSTM_OK; }
    s->cnt_words = (size_t)n * CNT_PER_LAYER + 16;
    if (cudaMalloc((void **)&s->cnt, s->cnt_words * sizeof(unsigned)) != cudaSuccess) { stack_small_destroy(s); return QLSTM_ERR_NOMEM; }
    s->owned.push_back(s->cnt);
    if (cudaMalloc((void **)&s->layers_dev, sizeof(SkLayer) * n) != cudaSuccess) { stack_small_destroy(s); return QLSTM_ERR_NOMEM; }
    s->owned.push_back(s->layers_dev);
    if (cudaMemcpy(s->layers_dev, s->layers.data(), sizeof(SkLayer) * n, cudaMemcpyHostToDevice) != cudaSuccess) {
        stack_small_destroy(s);
        return QLSTM_ERR_CUDA;
    }
    for (int NB : {1, 2, 4}) {
        if (cudaFuncSetAttribute(sk_kernel(NB), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s->smem) != cudaSuccess) {
            stack_small_destroy(s);
            return QLSTM_OK;
        }
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sk_kernel(NB), SK_THREADS, s->smem) != cudaSuccess || per_sm < 1) {
            stack_small_destroy(s);
            return QLSTM_OK;
        }
    }
    s->ok = true;
    *out = s;
    return QLSTM_OK;
}

bool stack_small_supported(const StackSmall *s, int T, int B) { return s && s->ok && B >= 1 && B <= s->max_B && T >= 1 && T <= s->max_T; }

void stack_small_debug_timeout(StackSmall *s, unsigned missing_arrivals, unsigned long long limit_ns)
{
    if (!s) return;
    s->dbg_missing = missing_arrivals;
    s->dbg_limit_ns = missing_arrivals ? limit_ns : 0;
}

int stack_small_groups(const StackSmall *s, int *blocks_per_layer)
{
    if (!s || !s->ok) return 0;
    if (blocks_per_layer) *blocks_per_layer = s->layers.empty() ? 0 : s->layers[0].n_cta;
    return s->n_layers;
}

int launch_stack_small(const StackSmall *s, const int8_t *x, int T, int B, int8_t *h, int16_t *c, int8_t *y, int *status,
                       cudaStream_t st)
{
    SkCall k;
    memset(&k, 0, sizeof(k));
    k.T = T; k.B = B; k.n_layers = s->n_layers;
    k.x = x; k.h = h; k.c = c; k.y = y;
    k.cnt = s->cnt;
    k.abort_word = s->cnt + (size_t)s->n_layers * CNT_PER_LAYER;
    k.status = status;
    k.wait_limit_ns = s->dbg_limit_ns ? s->dbg_limit_ns : SK_WAIT_LIMIT_NS;
    k.missing_arrivals = s->dbg_missing;
    if (cudaMemsetAsync(s->cnt, 0, s->cnt_words * sizeof(unsigned), st) != cudaSuccess) return QLSTM_ERR_CUDA;
    const int NB = B == 1 ? 1 : (B == 2 ? 2 : 4);
    const SkLayer *layers = s->layers_dev;
    void *args[] = {(void *)&layers, (void *)&k};
    cudaError_t e = cudaLaunchCooperativeKernel(sk_kernel(NB), dim3(s->grid), dim3(SK_THREADS), args, s->smem, st);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return e == cudaErrorCooperativeLaunchTooLarge ? QLSTM_ERR_LAUNCH : QLSTM_ERR_CUDA;
    }
    return QLSTM_OK;
}

}  // namespace ql
