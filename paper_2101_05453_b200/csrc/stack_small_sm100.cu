// Whole-stack kernel for small batches (up to 16 rows): every layer and every time step in ONE cooperative launch.
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
#include <algorithm>
#include <cstring>
#include <vector>

#include "../../include/qlstm.h"
#include "fast_kernels.h"

namespace ql {

namespace {

constexpr int SK_THREADS = 512;              // 128 registers per thread: the mat-vec loops keep two rows of weight loads in flight
constexpr int SK_WARPS = SK_THREADS / 32;
constexpr unsigned long long SK_WAIT_LIMIT_NS = 2000000000ull;     // 2 s per wait

// counters of one layer (monotonic over a call): arrivals after the gate sums (layer norm), after the output gate's
// sums (layer norm + peephole), after the hidden state (projection), and at the end of a step
enum { CNT_A = 0, CNT_A2 = 1, CNT_M = 2, CNT_H = 3, CNT_PER_LAYER = 16 };      // 64 bytes apart

struct SkLayer {
    int I, C, O, G, N;
    DivMagic div_c;                // division by C (layer-norm statistics) as a multiplication
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
    unsigned *cnt_next;            // the other set of counters (and abort word): cleared by this call for the next one
    int cnt_words;
    int *status;
    unsigned long long wait_limit_ns;
    unsigned missing_arrivals;     // 0; a test makes every counter wait for arrivals that never come
    int sequential;                // schedule: 0 wavefront (one group of blocks per layer), 1 every layer on all blocks
    int max_I, max_O, max_C_proj, max_npc;   // widest layer: sizes of the shared-memory buffers
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

// Sums of NB values per lane over the gs lanes that share a row.  While a lane still holds more than one value a round
// halves what it keeps - it sends the half it gives up and adds the half it receives - so the rounds cost
// NB/2 + NB/4 + ... shuffles instead of NB each (the shuffle unit issues one per clock for the whole SM, and at 8 or 16
// batch rows it was the busiest unit of the mat-vecs).  Afterwards acc[0 .. cnt) of a lane with `emitter` set hold the
// sums of the batch rows b0 .. b0 + cnt - 1.
template <int NB, int S>
__device__ __forceinline__ void group_reduce_round(int32_t (&acc)[NB], int off, int lg, int &b0, bool &emitter)
{
    constexpr int CNT = (NB >> S) >= 1 ? (NB >> S) : 1;
    if (off < 1) return;
    if constexpr (CNT > 1) {
        const bool up = (lg & off) != 0;
#pragma unroll
        for (int i = 0; i < CNT / 2; ++i) {
            const int32_t keep = up ? acc[i + CNT / 2] : acc[i], give = up ? acc[i] : acc[i + CNT / 2];
            acc[i] = keep + __shfl_xor_sync(0xffffffffu, give, off);
        }
        if (up) b0 += CNT / 2;
    } else {
        acc[0] += __shfl_xor_sync(0xffffffffu, acc[0], off);
        if (lg & off) emitter = false;               // every lane of the pair holds the sum: one of them emits it
    }
}
template <int NB>
__device__ __forceinline__ int group_reduce(int32_t (&acc)[NB], int gs, int lg, int &b0, bool &emitter)
{
    b0 = 0;
    if constexpr (NB <= 2) {                         // too few values to share out: the plain butterfly, lane b emits row b
        for (int off = gs >> 1; off > 0; off >>= 1) {
#pragma unroll
            for (int b = 0; b < NB; ++b) acc[b] += __shfl_xor_sync(0xffffffffu, acc[b], off);
        }
        if (NB == 2 && gs > 1) {
            if (lg == 1) { acc[0] = acc[NB - 1]; b0 = 1; }
            emitter = lg < 2;
            return 1;
        }
        emitter = lg == 0;
        return NB;
    }
    emitter = true;
    group_reduce_round<NB, 0>(acc, gs >> 1, lg, b0, emitter);
    group_reduce_round<NB, 1>(acc, gs >> 2, lg, b0, emitter);
    group_reduce_round<NB, 2>(acc, gs >> 3, lg, b0, emitter);
    group_reduce_round<NB, 3>(acc, gs >> 4, lg, b0, emitter);
    group_reduce_round<NB, 4>(acc, gs >> 5, lg, b0, emitter);
    const int cnt = NB / gs;                         // gs and NB are powers of two
    return cnt >= 1 ? cnt : 1;
}

// rows [0, nrows) of a row-major int8 matrix (K bytes per row, K a multiple of 16) times NB vectors held in shared
// memory as [NB][K]; emit(row, b, acc) runs once per (row, b < NB) on one lane.  gs lanes share a row (a power of two
// that divides the number of 16-byte chunks of a row, so that every lane takes the same number of chunks CPL).
// A warp keeps the weight loads of two rows per lane in flight (R2): the loop is bound by the latency of those loads
// and by the shared-memory reads of the vectors, which the two rows share.
template <int NB, int CPL, bool R2, bool VG, class F>
__device__ __forceinline__ void matvec_rows_t(const int8_t *rows, int nrows, int K, int gs, const int8_t *vec_s, F emit)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lg = lane & (gs - 1), sub = lane / gs, rpw = 32 / gs;
    const int stride = SK_WARPS * rpw;
    constexpr int NR = R2 ? 2 : 1;
    for (int r0 = warp * rpw; r0 < nrows; r0 += stride * NR) {
        int32_t acc[NR][NB];
        uint4 w[NR][CPL];
        bool valid[NR];
#pragma unroll
        for (int q = 0; q < NR; ++q) {
            const int r = r0 + q * stride + sub;
            valid[q] = r < nrows;
            const uint4 *wp = reinterpret_cast<const uint4 *>(rows + (size_t)(valid[q] ? r : 0) * K) + lg;
#pragma unroll
            for (int j = 0; j < CPL; ++j) w[q][j] = valid[q] ? ld_stream(wp + j * gs) : make_uint4(0, 0, 0, 0);   // all loads in flight
        }
        // VG: the vectors are read straight from global memory (L2: other blocks wrote them this step), their loads in
        // flight together with the weights' - at one batch row this saves the round trip of staging them first
        uint4 vg[VG ? CPL : 1][VG ? NB : 1];
        if (VG) {
#pragma unroll
            for (int j = 0; j < CPL; ++j)
#pragma unroll
                for (int b = 0; b < NB; ++b) vg[VG ? j : 0][VG ? b : 0] = __ldcg(reinterpret_cast<const uint4 *>(vec_s + (size_t)b * K) + lg + j * gs);
        }
#pragma unroll
        for (int q = 0; q < NR; ++q)
#pragma unroll
            for (int b = 0; b < NB; ++b) acc[q][b] = 0;
        // every vector chunk is read once and used for both rows
#pragma unroll
        for (int j = 0; j < CPL; ++j) {
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                const uint4 v = VG ? vg[VG ? j : 0][VG ? b : 0] : reinterpret_cast<const uint4 *>(vec_s + (size_t)b * K)[lg + j * gs];
#pragma unroll
                for (int q = 0; q < NR; ++q) {
                    acc[q][b] = __dp4a((int)w[q][j].x, (int)v.x, acc[q][b]);
                    acc[q][b] = __dp4a((int)w[q][j].y, (int)v.y, acc[q][b]);
                    acc[q][b] = __dp4a((int)w[q][j].z, (int)v.z, acc[q][b]);
                    acc[q][b] = __dp4a((int)w[q][j].w, (int)v.w, acc[q][b]);
                }
            }
        }
#pragma unroll
        for (int q = 0; q < NR; ++q) {
            int b0;
            bool emitter;
            const int cnt = group_reduce<NB>(acc[q], gs, lg, b0, emitter);      // the lanes of a row share out the batch rows
            if (valid[q] && emitter) {
#pragma unroll
                for (int i = 0; i < NB; ++i)
                    if (i < cnt) emit(r0 + q * stride + sub, b0 + i, acc[q][i]);
            }
        }
    }
}

// any number of chunks per lane: one load at a time, four trips unrolled
template <int NB, bool VG, class F>
__device__ __forceinline__ void matvec_rows_any(const int8_t *rows, int nrows, int K, int gs, const int8_t *vec_s, F emit)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lg = lane & (gs - 1), sub = lane / gs, rpw = 32 / gs;
    const int cpl = (K >> 4) / gs;
    for (int r0 = warp * rpw; r0 < nrows; r0 += SK_WARPS * rpw) {
        const int r = r0 + sub;
        const bool valid = r < nrows;
        int32_t acc[NB];
#pragma unroll
        for (int b = 0; b < NB; ++b) acc[b] = 0;
        if (valid) {
            const uint4 *wp = reinterpret_cast<const uint4 *>(rows + (size_t)r * K) + lg;
#pragma unroll 4
            for (int j = 0; j < cpl; ++j) {
                const uint4 w = ld_stream(wp + j * gs);
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const uint4 *vp = reinterpret_cast<const uint4 *>(vec_s + (size_t)b * K) + lg + j * gs;
                    const uint4 v = VG ? __ldcg(vp) : *vp;
                    acc[b] = __dp4a((int)w.x, (int)v.x, acc[b]);
                    acc[b] = __dp4a((int)w.y, (int)v.y, acc[b]);
                    acc[b] = __dp4a((int)w.z, (int)v.z, acc[b]);
                    acc[b] = __dp4a((int)w.w, (int)v.w, acc[b]);
                }
            }
        }
        int b0;
        bool emitter;
        const int cnt = group_reduce<NB>(acc, gs, lg, b0, emitter);
        if (valid && emitter) {
#pragma unroll
            for (int i = 0; i < NB; ++i)
                if (i < cnt) emit(r, b0 + i, acc[i]);
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

template <int NB, bool VG, class F>
__device__ __forceinline__ void matvec_rows(const int8_t *rows, int nrows, int K, const int8_t *vec, F emit)
{
    const int gs = lanes_per_row(K);
    constexpr bool R2 = NB <= 8;             // sixteen batch rows: the accumulators of two rows would not fit in registers
    switch ((K >> 4) / gs) {
        case 1: matvec_rows_t<NB, 1, R2, VG>(rows, nrows, K, gs, vec, emit); break;
        case 2: matvec_rows_t<NB, 2, R2, VG>(rows, nrows, K, gs, vec, emit); break;
        case 4: matvec_rows_t<NB, 4, R2, VG>(rows, nrows, K, gs, vec, emit); break;
        case 5: matvec_rows_t<NB, 5, R2, VG>(rows, nrows, K, gs, vec, emit); break;
        default: matvec_rows_any<NB, VG>(rows, nrows, K, gs, vec, emit); break;
    }
}

// The B vectors of a mat-vec, [B][K] int8 in global memory.  With one batch row they are read in place (when 16-byte
// aligned); otherwise they are staged in shared memory first, rows >= B zero.
template <int NB, class F>
__device__ __forceinline__ void matvec_with(const int8_t *rows, int nrows, int K, const int8_t *vec_g, int B, int8_t *stage_s,
                                            bool written_by_other_blocks, F emit)
{
    if (NB == 1 && (((uintptr_t)vec_g) & 15) == 0) {
        matvec_rows<NB, true>(rows, nrows, K, vec_g, emit);
        return;
    }
    if (written_by_other_blocks) stage_vec(stage_s, vec_g, B, NB, K);
    else stage_vec_bytes(stage_s, vec_g, B, NB, K);
    __syncthreads();
    matvec_rows<NB, false>(rows, nrows, K, stage_s, emit);
}

// What a block does for one layer: its share of the cells and of the projection rows, and where things live.
struct Role {
    const SkLayer *L;              // shared memory
    int li, rank;
    int u0, cells, npc, n0, n_cnt; // own cells and gate rows
    int p_lo, p_cnt;               // own projection rows
    int16_t *c_s;                  // [NB][cpc] cell state, resident over the call
    // per-row constants of the block's own rows, copied to shared memory once (a global load inside every epilogue
    // would be one more round trip in each step's chain): indexed by the local gate row / projection row
    const int32_t *bx, *bh, *bln, *bp;
    const int16_t *Lw, *Pw;
    unsigned *cnt;                 // the layer's counters
    const unsigned *cnt_below;     // CNT_H of the layer below, or null
    unsigned n_below;
    const int8_t *in_seq;          // [T][B][I]
    int8_t *out_seq;               // [T][B][O]
    int8_t *h_state;
    int16_t *c_state;
};

struct SkSmem {
    int8_t *x_s, *h_s, *m_s;       // staged operands [NB][I], [NB][O], [NB][C]
    int16_t *xs_s, *hs_s;          // [NB][npc] rescaled input and recurrent terms
    int16_t *pre_s;                // [NB][npc] gate sums
    LnRow *ln_s;                   // [NB][4]
};

// ---- the pieces of one layer-step -------------------------------------------------------------------------------

// input term (Section 3.2.4, first rescale): xs = sat16(rescale(W x_t + bx, eff_x))
template <int NB>
__device__ __forceinline__ void input_term(const SkCall &k, const Role &r, const SkSmem &s, int t)
{
    const SkLayer &L = *r.L;
    const int B = k.B, npc = r.npc, n0 = r.n0, G = L.G;
    matvec_with<NB>(L.W + (size_t)n0 * L.I, r.n_cnt, L.I, r.in_seq + (size_t)t * B * L.I, B, s.x_s, true, [&](int n, int b, int32_t acc) {
        if (b < B) s.xs_s[b * npc + n] = (int16_t)sat16(sk_rescale(acc + r.bx[n], L.eff_x[n % G]));
    });
}

// recurrent term: hs = sat16(rescale(sat32(R h^{t-1} + bh), eff_h)); h^{t-1} is the previous row block of the layer's
// output sequence (the caller's h at t = 0)
template <int NB>
__device__ __forceinline__ void recurrent_term(const SkCall &k, const Role &r, const SkSmem &s, int t)
{
    const SkLayer &L = *r.L;
    const int B = k.B, npc = r.npc, n0 = r.n0, G = L.G;
    const int8_t *h_prev = t == 0 ? r.h_state : r.out_seq + (size_t)(t - 1) * B * L.O;
    matvec_with<NB>(L.R + (size_t)n0 * L.O, r.n_cnt, L.O, h_prev, B, s.h_s, t != 0, [&](int n, int b, int32_t acc) {
        if (b < B) s.hs_s[b * npc + n] = (int16_t)sat16(sk_rescale(sk_add_sat(acc, r.bh[n]), L.eff_h[n % G]));
    });
}

// Warp-wide sums of the layer-norm statistics with the 32-bit hardware reduction (one instruction, where a shuffle
// tree of a 64-bit value is ten): a sum of at most a row of int16 values fits 32 bits on every lane and in total; a sum
// of squares (non-negative, below 2^44 in total) goes as its low 20 bits and the rest.  Every lane gets the result.
__device__ __forceinline__ long long warp_sum_small(long long v) { return (long long)__reduce_add_sync(0xffffffffu, (int)v); }
__device__ __forceinline__ long long warp_sum_nonneg(long long v)
{
    const unsigned long long q = (unsigned long long)v;
    const unsigned lo = __reduce_add_sync(0xffffffffu, (unsigned)(q & 0xfffffu));
    const unsigned hi = __reduce_add_sync(0xffffffffu, (unsigned)(q >> 20));
    return (long long)(((unsigned long long)hi << 20) + lo);
}

// layer-norm constants of the rows for the gate slots in `slots`: the block's per-row sums go to global memory, the
// group meets, every block adds the group's shares (integer sums: the order does not matter)
__device__ __forceinline__ bool exchange_stats(const SkCall &k, const Role &r, const SkSmem &s, int round, unsigned slots,
                                               unsigned *counter, unsigned target, int *abort_s)
{
    const SkLayer &L = *r.L;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, B = k.B, G = L.G;
    long long *mine = L.part + ((size_t)r.rank * 2 + round) * B * 8;
    for (int task = warp; task < B * 4; task += SK_WARPS) {
        const int b = task >> 2, gi = task & 3;
        if (!((slots >> gi) & 1u)) continue;
        long long sum = 0, sq = 0;
        for (int ul = lane; ul < r.cells; ul += 32) {
            const int32_t v = s.pre_s[b * r.npc + ul * G + gi];
            sum += v;
            sq += (long long)(v * v);
        }
        sum = warp_sum_small(sum);
        sq = warp_sum_nonneg(sq);
        if (lane == 0) { mine[task * 2] = sum; mine[task * 2 + 1] = sq; }
    }
    sk_arrive(counter);
    if (!sk_wait(k, counter, target, abort_s)) return false;
    for (int task = warp; task < B * 4; task += SK_WARPS) {
        const int gi = task & 3;
        if (!((slots >> gi) & 1u)) continue;
        long long sum = 0, sq = 0;
        for (int q = lane; q < L.n_cta; q += 32) {
            const long long *share = L.part + ((size_t)q * 2 + round) * B * 8 + task * 2;
            sum += __ldcg(share);
            sq += __ldcg(share + 1);
        }
        sum = warp_sum_small(sum);
        sq = warp_sum_nonneg(sq);
        if (lane == 0) s.ln_s[task] = make_ln_row(ln_stats_fast(sum, sq, L.div_c));
    }
    __syncthreads();
    return true;
}

// everything of step t after the two terms; ends with the block's arrival on the layer's step counter
template <int NB>
__device__ __forceinline__ bool finish_step(const SkCall &k, const Role &r, const SkSmem &s, int t, int *abort_s)
{
    const SkLayer &L = *r.L;
    const int B = k.B, G = L.G, C = L.C, O = L.O, npc = r.npc, cells = r.cells, u0 = r.u0, cpc = L.cpc;
    const bool proj = (L.flags & F_PROJECTION) != 0, ln = (L.flags & F_LAYERNORM) != 0, peep = (L.flags & F_PEEPHOLE) != 0;
    const int SF = (G == 4) ? 1 : 0, SZ = SF + 1, SO = SF + 2;
    const unsigned n_grp = (unsigned)L.n_cta;
    __syncthreads();
    // gate sums (Section 3.2.4 / 3.2.5): X + H (+ peephole on c^{t-1} for the input and forget gates); with a peephole the
    // output gate's sum waits for c^t (Eq. 5)
    for (int i = threadIdx.x; i < B * r.n_cnt; i += SK_THREADS) {
        const int b = i / r.n_cnt, n = i - b * r.n_cnt, gi = n % G, ul = n / G;
        int32_t v = (int32_t)s.xs_s[b * npc + n] + (int32_t)s.hs_s[b * npc + n];
        if (peep && gi == SO) continue;
        if (peep && gi != SZ) v += sat16(sk_rescale((int32_t)r.Pw[n] * r.c_s[b * cpc + ul], L.eff_c[gi]));
        s.pre_s[b * npc + n] = (int16_t)sat16(v);
    }
    __syncthreads();
    if (ln) {
        const unsigned all = (1u << G) - 1u;
        if (!exchange_stats(k, r, s, 0, peep ? (all & ~(1u << SO)) : all, r.cnt + CNT_A, (unsigned)(t + 1) * n_grp, abort_s)) return false;
    }
    const bool quad = B * cells * 4 <= SK_THREADS;
    if (quad) {
        // Few cells (one or two batch rows): four lanes per cell, one gate each, so that the cell's five nonlinearities
        // are not one thread's serial chain.  Lane j takes gate slot j (layer norm + sigmoid / tanh), the group exchanges
        // the gate values with shuffles, every lane forms c^t, then the output gate's lane and the update gate's lane
        // compute sigmoid(o) and tanh(c^t) side by side and lane 0 forms the hidden state.
        const int task_i = threadIdx.x >> 2, j = threadIdx.x & 3, base = (threadIdx.x & 31) & ~3;
        const bool task = task_i < B * cells;
        const int b = task ? task_i / cells : 0, ul = task ? task_i - b * cells : 0;
        const int nl = ul * G;
        const bool mine = task && j < G;                           // this lane has a gate
        auto gate_in_of = [&](int g) -> int32_t {
            const int32_t v = s.pre_s[b * npc + nl + g];
            return ln ? ln_apply_fast(v, s.ln_s[b * 4 + g], r.Lw[nl + g], r.bln[nl + g], L.eff_ln[g], make_fast_scale(L.eff_ln[g])) : v;
        };
        int32_t val = 0;
        if (mine && !(peep && j == SO)) {
            const int32_t v = gate_in_of(j);
            val = (j == SZ) ? tanh_q_fast(v, 3) : sigmoid_q_fast(v, 3);
        }
        const int32_t f = __shfl_sync(0xffffffffu, val, base + SF), z = __shfl_sync(0xffffffffu, val, base + SZ);
        int32_t ig = __shfl_sync(0xffffffffu, val, base);
        int32_t o = __shfl_sync(0xffffffffu, val, base + SO);
        if (G != 4) { ig = 32768 - f; if (ig > 32767) ig = 32767; }  // coupled input gate, Section 3.2.9
        const int32_t c_old = task ? r.c_s[b * cpc + ul] : 0;
        const int32_t c_new = cell_update_fast(ig, z, f, c_old, L.m_bits);
        __syncwarp();
        if (task && j == 0) r.c_s[b * cpc + ul] = (int16_t)c_new;
        if (peep && task && j == SO) {
            const int32_t ao = sat16((int32_t)s.xs_s[b * npc + nl + SO] + (int32_t)s.hs_s[b * npc + nl + SO] +
                                     sat16(sk_rescale((int32_t)r.Pw[nl + SO] * c_new, L.eff_c[SO])));
            if (ln) s.pre_s[b * npc + nl + SO] = (int16_t)ao;     // waits for the row's statistics
            else val = sigmoid_q_fast(ao, 3);
        }
        if (ln && peep) {
            __syncthreads();
            if (!exchange_stats(k, r, s, 1, 1u << SO, r.cnt + CNT_A2, (unsigned)(t + 1) * n_grp, abort_s)) return false;
            if (task && j == SO) val = sigmoid_q_fast(gate_in_of(SO), 3);
        }
        if (peep) o = __shfl_sync(0xffffffffu, val, base + SO);
        int32_t tc = (task && j == SZ) ? tanh_q_fast(c_new, L.m_bits) : 0;
        tc = __shfl_sync(0xffffffffu, tc, base + SZ);
        if (task && j == 0) {
            const int32_t mq = sat8(sk_rescale(o * tc, L.eff_m) + L.zp_m);              // Section 3.2.7
            if (proj) L.m[(size_t)b * C + u0 + ul] = (int8_t)mq;
            else r.out_seq[((size_t)t * B + b) * O + u0 + ul] = (int8_t)mq;
        }
    } else {
        // elementwise, one cell per thread
        for (int i = threadIdx.x; i < B * cells; i += SK_THREADS) {
            const int b = i / cells, ul = i - b * cells;
            const int nl = ul * G;
            const int16_t *pre = s.pre_s + b * npc + nl;
            const LnRow *lr = s.ln_s + b * 4;
            // input of the nonlinearity of gate slot g: the gate sum, after layer norm when the layer has it
            auto gate_in = [&](int g) -> int32_t {
                const int32_t v = pre[g];
                return ln ? ln_apply_fast(v, lr[g], r.Lw[nl + g], r.bln[nl + g], L.eff_ln[g], make_fast_scale(L.eff_ln[g])) : v;
            };
            const int32_t f = sigmoid_q_fast(gate_in(SF), 3), z = tanh_q_fast(gate_in(SZ), 3);
            int32_t ig;
            if (G == 4) ig = sigmoid_q_fast(gate_in(0), 3);
            else { ig = 32768 - f; if (ig > 32767) ig = 32767; }    // coupled input gate, Section 3.2.9
            const int32_t c_old = r.c_s[b * cpc + ul];
            const int32_t c_new = cell_update_fast(ig, z, f, c_old, L.m_bits);
            r.c_s[b * cpc + ul] = (int16_t)c_new;
            int32_t ao;
            if (peep) {
                ao = sat16((int32_t)s.xs_s[b * npc + nl + SO] + (int32_t)s.hs_s[b * npc + nl + SO] +
                           sat16(sk_rescale((int32_t)r.Pw[nl + SO] * c_new, L.eff_c[SO])));
                if (ln) { s.pre_s[b * npc + nl + SO] = (int16_t)ao; continue; }      // waits for the row's statistics
            } else {
                ao = gate_in(SO);
            }
            const int32_t mq = hidden_q_fast(sigmoid_q_fast(ao, 3), c_new, L.m_bits, L.eff_m, make_fast_scale(L.eff_m), L.zp_m);
            if (proj) L.m[(size_t)b * C + u0 + ul] = (int8_t)mq;
            else r.out_seq[((size_t)t * B + b) * O + u0 + ul] = (int8_t)mq;
        }
        if (ln && peep) {
            __syncthreads();
            if (!exchange_stats(k, r, s, 1, 1u << SO, r.cnt + CNT_A2, (unsigned)(t + 1) * n_grp, abort_s)) return false;
            for (int i = threadIdx.x; i < B * cells; i += SK_THREADS) {
                const int b = i / cells, ul = i - b * cells;
                const int n = ul * G + SO;                     // index into the block's own rows
                const int32_t ao = ln_apply_fast(s.pre_s[b * npc + ul * G + SO], s.ln_s[b * 4 + SO], r.Lw[n], r.bln[n], L.eff_ln[SO],
                                                 make_fast_scale(L.eff_ln[SO]));
                const int32_t mq = hidden_q_fast(sigmoid_q_fast(ao, 3), r.c_s[b * cpc + ul], L.m_bits, L.eff_m,
                                                 make_fast_scale(L.eff_m), L.zp_m);
                if (proj) L.m[(size_t)b * C + u0 + ul] = (int8_t)mq;
                else r.out_seq[((size_t)t * B + b) * O + u0 + ul] = (int8_t)mq;
            }
        }
    }
    // projection (Section 3.2.8): needs every m of the layer
    if (proj) {
        sk_arrive(r.cnt + CNT_M);
        if (!sk_wait(k, r.cnt + CNT_M, (unsigned)(t + 1) * n_grp, abort_s)) return false;
        const int p_lo = r.p_lo;
        int8_t *out = r.out_seq + (size_t)t * B * O;
        matvec_with<NB>(L.Wproj + (size_t)p_lo * C, r.p_cnt, C, L.m, B, s.m_s, true, [&](int row, int b, int32_t acc) {
            if (b < B) out[(size_t)b * O + p_lo + row] = (int8_t)sat8(sk_rescale(sk_add_sat(acc, r.bp[row]), L.eff_proj) + L.zp_h);
        });
    }
    // h^t is complete once every block of the group has arrived
    sk_arrive(r.cnt + CNT_H);
    return true;
}

// bytes a role keeps resident in shared memory: cell state [NB][cpc] int16, then bx, bh, bln [npc] int32, bp [rpc] int32,
// L, P [npc] int16
__host__ __device__ inline size_t role_bytes(int NB, int cpc, int G, int rpc)
{
    const size_t npc = (size_t)cpc * G;
    return (((size_t)NB * cpc * 2 + 15) & ~(size_t)15) + npc * 12 + (((size_t)rpc * 4 + 15) & ~(size_t)15) + ((npc * 4 + 15) & ~(size_t)15);
}

// calls of at least this many steps keep the per-row constants of a block's rows in shared memory
constexpr int SK_RESIDENT_MIN_T = 4;

__device__ __forceinline__ Role make_role(const SkCall &k, const SkLayer *Ls, int li, int rank, uint8_t *region, int NB)
{
    const SkLayer &L = Ls[li];
    Role r;
    r.L = &L; r.li = li; r.rank = rank;
    r.u0 = rank * L.cpc;
    r.cells = L.C - r.u0 < L.cpc ? L.C - r.u0 : L.cpc;
    if (r.cells < 0) r.cells = 0;
    r.npc = L.cpc * L.G; r.n0 = r.u0 * L.G; r.n_cnt = r.cells * L.G;
    r.p_lo = rank * L.rpc;
    r.p_cnt = (L.flags & F_PROJECTION) ? (L.O - r.p_lo < L.rpc ? L.O - r.p_lo : L.rpc) : 0;
    if (r.p_cnt < 0) r.p_cnt = 0;
    {
        uint8_t *p = region;
        r.c_s = (int16_t *)p;  p += ((size_t)NB * L.cpc * 2 + 15) & ~(size_t)15;
        if (k.T >= SK_RESIDENT_MIN_T) {
            r.bx = (const int32_t *)p;  p += (size_t)r.npc * 4;
            r.bh = (const int32_t *)p;  p += (size_t)r.npc * 4;
            r.bln = (const int32_t *)p; p += (size_t)r.npc * 4;
            r.bp = (const int32_t *)p;  p += ((size_t)L.rpc * 4 + 15) & ~(size_t)15;
            r.Lw = (const int16_t *)p;  p += (size_t)r.npc * 2;
            r.Pw = (const int16_t *)p;
        } else {                                               // a call of a few steps reads them where they are
            r.bx = L.bx + r.n0; r.bh = L.bh + r.n0;
            r.bln = L.bln ? L.bln + r.n0 : nullptr;
            r.bp = L.bp ? L.bp + r.p_lo : nullptr;
            r.Lw = L.L ? L.L + r.n0 : nullptr;
            r.Pw = L.P ? L.P + r.n0 : nullptr;
        }
    }
    r.cnt = k.cnt + (size_t)li * CNT_PER_LAYER;
    r.cnt_below = li > 0 ? k.cnt + (size_t)(li - 1) * CNT_PER_LAYER + CNT_H : nullptr;
    r.n_below = li > 0 ? (unsigned)Ls[li - 1].n_cta : 0u;
    r.in_seq = li > 0 ? Ls[li - 1].seq : k.x;
    r.out_seq = L.seq ? L.seq : k.y;
    r.h_state = k.h + L.h_off * k.B;
    r.c_state = k.c + L.c_off * k.B;
    return r;
}

// all threads: the per-row constants of a role's own rows into its shared-memory region
__device__ __forceinline__ void load_role_consts(const Role &r)
{
    const SkLayer &L = *r.L;
    if (r.bx == L.bx + r.n0) return;                           // not resident for this call
    const bool ln = (L.flags & F_LAYERNORM) != 0, peep = (L.flags & F_PEEPHOLE) != 0;
    for (int n = threadIdx.x; n < r.n_cnt; n += SK_THREADS) {
        const_cast<int32_t *>(r.bx)[n] = L.bx[r.n0 + n];
        const_cast<int32_t *>(r.bh)[n] = L.bh[r.n0 + n];
        const_cast<int32_t *>(r.bln)[n] = ln ? L.bln[r.n0 + n] : 0;
        const_cast<int16_t *>(r.Lw)[n] = ln ? L.L[r.n0 + n] : (int16_t)0;
        const_cast<int16_t *>(r.Pw)[n] = peep ? L.P[r.n0 + n] : (int16_t)0;
    }
    for (int q = threadIdx.x; q < r.p_cnt; q += SK_THREADS) const_cast<int32_t *>(r.bp)[q] = L.bp[r.p_lo + q];
}

// Two schedules, chosen by the host per call:
//   wavefront   one group of blocks per layer; group l works on step t while group l + 1 works on step t - 1.  Between
//               its arrival at the end of step t and the wait for the group, a block already computes the input term of
//               step t + 1 (which needs the layer below, not the block's own group).
//   sequential  every layer on all blocks, one layer after the other (calls of a few steps: there is nothing to
//               overlap across steps, and a layer gets the whole machine's bandwidth).  Between its arrival at the end
//               of layer l and the wait, a block already computes the recurrent term of layer l + 1 (which needs that
//               layer's own h^{t-1}, not layer l).
template <int NB>
__global__ void __launch_bounds__(SK_THREADS, 1) k_stack_small(const SkLayer *__restrict__ layers, SkCall k)
{
    extern __shared__ __align__(16) uint8_t sk_smem[];
    __shared__ int abort_s;
    const int cta = blockIdx.x, nl = k.n_layers, B = k.B, T = k.T;
    // the layer descriptions, then the buffers (sized for the widest layer), then the cell states
    SkLayer *Ls = reinterpret_cast<SkLayer *>(sk_smem);
    for (int i = threadIdx.x; i < (int)(nl * sizeof(SkLayer) / 4); i += SK_THREADS)
        reinterpret_cast<uint32_t *>(Ls)[i] = reinterpret_cast<const uint32_t *>(layers)[i];
    if (threadIdx.x == 0) abort_s = 0;
    if (cta == 0) {
        // calls alternate between two sets of counters; nothing in this call touches the other one, so it is cleared here
        // for the next call (no memset launch per call: a one-step call is only a hundred-odd microseconds long)
        for (int i = threadIdx.x; i < k.cnt_words; i += SK_THREADS) k.cnt_next[i] = 0u;
        if (threadIdx.x == 0) *k.status = 0;
    }
    __syncthreads();
    SkSmem s;
    uint8_t *c_base;                                           // resident regions of the roles
    {
        uint8_t *p = sk_smem + (((size_t)nl * sizeof(SkLayer) + 15) & ~(size_t)15);
        s.x_s = (int8_t *)p;  p += (size_t)NB * k.max_I;
        s.h_s = (int8_t *)p;  p += (size_t)NB * k.max_O;
        s.m_s = (int8_t *)p;  p += (size_t)NB * k.max_C_proj;
        s.ln_s = (LnRow *)p;  p += (size_t)NB * 4 * sizeof(LnRow);
        s.xs_s = (int16_t *)p; p += (size_t)NB * k.max_npc * 2;
        s.hs_s = (int16_t *)p; p += (size_t)NB * k.max_npc * 2;
        s.pre_s = (int16_t *)p; p += (size_t)NB * k.max_npc * 2;
        c_base = (uint8_t *)(((uintptr_t)p + 15) & ~(uintptr_t)15);
    }
    bool ok = true;

    if (!k.sequential) {
        int li = -1;
        for (int l = 0; l < nl; ++l)
            if (cta >= Ls[l].cta0 && cta < Ls[l].cta0 + Ls[l].n_cta) li = l;
        if (li < 0) return;                                    // spare block: takes no part in any counter
        const Role r = make_role(k, Ls, li, cta - Ls[li].cta0, c_base, NB);
        load_role_consts(r);
        const unsigned n_grp = (unsigned)r.L->n_cta;
        for (int i = threadIdx.x; i < B * r.cells; i += SK_THREADS) {
            const int b = i / r.cells, ul = i - b * r.cells;
            r.c_s[b * r.L->cpc + ul] = r.c_state[(size_t)b * r.L->C + r.u0 + ul];
        }
        __syncthreads();
        if (r.cnt_below) ok = sk_wait(k, r.cnt_below, r.n_below, &abort_s);
        if (ok) input_term<NB>(k, r, s, 0);
        for (int t = 0; t < T && ok; ++t) {
            recurrent_term<NB>(k, r, s, t);
            ok = finish_step<NB>(k, r, s, t, &abort_s);
            if (!ok) break;
            if (t + 1 < T) {
                if (r.cnt_below) ok = sk_wait(k, r.cnt_below, (unsigned)(t + 2) * r.n_below, &abort_s);
                if (!ok) break;
                input_term<NB>(k, r, s, t + 1);
            }
            ok = sk_wait(k, r.cnt + CNT_H, (unsigned)(t + 1) * n_grp, &abort_s);
        }
        if (ok) {
            for (int i = threadIdx.x; i < B * r.cells; i += SK_THREADS) {
                const int b = i / r.cells, ul = i - b * r.cells;
                r.c_state[(size_t)b * r.L->C + r.u0 + ul] = r.c_s[b * r.L->cpc + ul];
            }
            if (T > 0) {
                // every block copies its share of the columns of h = the last row block of the output sequence
                const int O = r.L->O, per = (O + r.L->n_cta - 1) / r.L->n_cta, o_lo = r.rank * per;
                const int o_hi = o_lo + per < O ? o_lo + per : O;
                for (int b = 0; b < B; ++b)
                    for (int o = o_lo + (int)threadIdx.x; o < o_hi; o += SK_THREADS)
                        r.h_state[(size_t)b * O + o] = __ldcg(r.out_seq + ((size_t)(T - 1) * B + b) * O + o);
            }
        }
    } else {
        // cell states of this block's cells of every layer
        size_t c_off = 0;
        for (int l = 0; l < nl; ++l) {
            const Role r = make_role(k, Ls, l, cta, c_base + c_off, NB);
            load_role_consts(r);
            for (int i = threadIdx.x; i < B * r.cells; i += SK_THREADS) {
                const int b = i / r.cells, ul = i - b * r.cells;
                r.c_s[b * r.L->cpc + ul] = r.c_state[(size_t)b * r.L->C + r.u0 + ul];
            }
            c_off += role_bytes(NB, Ls[l].cpc, Ls[l].G, Ls[l].rpc);
        }
        __syncthreads();
        for (int t = 0; t < T && ok; ++t) {
            c_off = 0;
            for (int l = 0; l < nl && ok; ++l) {
                const Role r = make_role(k, Ls, l, cta, c_base + c_off, NB);
                c_off += role_bytes(NB, Ls[l].cpc, Ls[l].G, Ls[l].rpc);
                const unsigned n_grp = (unsigned)r.L->n_cta;
                // this layer's own h^{t-1} (complete long ago for every layer but the last)
                if (t > 0) ok = sk_wait(k, r.cnt + CNT_H, (unsigned)t * n_grp, &abort_s);
                if (!ok) break;
                recurrent_term<NB>(k, r, s, t);
                // the layer below at this step: its arrival was the last thing this block did
                if (r.cnt_below) ok = sk_wait(k, r.cnt_below, (unsigned)(t + 1) * r.n_below, &abort_s);
                if (!ok) break;
                input_term<NB>(k, r, s, t);
                ok = finish_step<NB>(k, r, s, t, &abort_s);
            }
        }
        // every layer's last step complete before the state goes back
        for (int l = 0; l < nl && ok; ++l)
            ok = sk_wait(k, k.cnt + (size_t)l * CNT_PER_LAYER + CNT_H, (unsigned)T * (unsigned)Ls[l].n_cta, &abort_s);
        if (ok) {
            c_off = 0;
            for (int l = 0; l < nl; ++l) {
                const Role r = make_role(k, Ls, l, cta, c_base + c_off, NB);
                c_off += role_bytes(NB, Ls[l].cpc, Ls[l].G, Ls[l].rpc);
                for (int i = threadIdx.x; i < B * r.cells; i += SK_THREADS) {
                    const int b = i / r.cells, ul = i - b * r.cells;
                    r.c_state[(size_t)b * r.L->C + r.u0 + ul] = r.c_s[b * r.L->cpc + ul];
                }
                if (T > 0) {
                    const int O = r.L->O, per = (O + r.L->n_cta - 1) / r.L->n_cta, o_lo = r.rank * per;
                    const int o_hi = o_lo + per < O ? o_lo + per : O;
                    for (int b = 0; b < B; ++b)
                        for (int o = o_lo + (int)threadIdx.x; o < o_hi; o += SK_THREADS)
                            r.h_state[(size_t)b * O + o] = __ldcg(r.out_seq + ((size_t)(T - 1) * B + b) * O + o);
                }
            }
        }
    }
    if (!ok && threadIdx.x == 0) atomicExch(k.status, 2);
}

}  // namespace

struct StackSmall {
    bool ok = false;
    int n_layers = 0, grid = 0, max_T = 0, max_B = 0;
    size_t smem = 0;
    SkLayer *plan_dev[2] = {nullptr, nullptr};     // [0] wavefront, [1] sequential
    std::vector<SkLayer> plan[2];
    int max_I = 0, max_O = 0, max_C_proj = 0, max_npc = 0;
    std::vector<void *> owned;
    unsigned *cnt = nullptr;       // two sets of counters + abort word, used by alternate calls
    size_t cnt_words = 0;          // words of one set
    unsigned calls = 0;
    unsigned dbg_missing = 0;
    unsigned long long dbg_limit_ns = 0;
};

static const void *sk_kernel(int NB)
{
    switch (NB) {
        case 1: return (const void *)k_stack_small<1>;
        case 2: return (const void *)k_stack_small<2>;
        case 4: return (const void *)k_stack_small<4>;
        case 8: return (const void *)k_stack_small<8>;
        default: return (const void *)k_stack_small<16>;
    }
}
static int sk_rows(int B) { return B <= 1 ? 1 : B <= 2 ? 2 : B <= 4 ? 4 : B <= 8 ? 8 : 16; }

void stack_small_destroy(StackSmall *s)
{
    if (!s) return;
    for (void *p : s->owned) cudaFree(p);
    delete s;
}

// shared memory of a block for NB batch rows under both schedules
static size_t sk_smem_bytes(const StackSmall &s, int NB)
{
    size_t common = (((size_t)s.n_layers * sizeof(SkLayer) + 15) & ~(size_t)15) + (size_t)NB * (s.max_I + s.max_O + s.max_C_proj) +
                    (size_t)NB * 4 * sizeof(LnRow) + 3 * (size_t)NB * s.max_npc * 2;
    size_t c_wave = 0, c_seq = 0;
    for (const SkLayer &L : s.plan[0]) c_wave = std::max(c_wave, role_bytes(NB, L.cpc, L.G, L.rpc));
    for (const SkLayer &L : s.plan[1]) c_seq += role_bytes(NB, L.cpc, L.G, L.rpc);
    return common + std::max(c_wave, c_seq) + 96;
}

// Plans the whole-stack kernel for a handle; *out stays null when the stack does not qualify (the per-layer kernels
// then run).  max_B beyond STACK_SMALL_MAX_B is fine: the kernel is only used for smaller batches.
int stack_small_create(const std::vector<const LayerParams *> &lp, int max_T, int max_B, int sm_count, StackSmall **out)
{
    *out = nullptr;
    const int n = (int)lp.size();
    if (n < 1 || n > sm_count || n > 64) return QLSTM_OK;
    for (const LayerParams *p : lp)
        if (p->I % 16 != 0 || p->O % 16 != 0 || p->C % 16 != 0) return QLSTM_OK;
    StackSmall *s = new StackSmall();
    s->n_layers = n;
    s->grid = sm_count;
    s->max_T = max_T;
    s->max_B = max_B < STACK_SMALL_MAX_B ? max_B : STACK_SMALL_MAX_B;
    int dev = 0, max_smem = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    auto fail = [&](int rc) { stack_small_destroy(s); return rc; };
    auto dalloc = [&](size_t bytes) -> void * {
        void *d = nullptr;
        if (cudaMalloc(&d, bytes ? bytes : 16) != cudaSuccess) return nullptr;
        s->owned.push_back(d);
        return d;
    };
    size_t h_off = 0, c_off = 0;
    for (int l = 0; l < n; ++l) {
        const LayerParams &p = *lp[l];
        SkLayer L;
        memset(&L, 0, sizeof(L));
        L.I = p.I; L.C = p.C; L.O = p.O; L.G = p.G; L.N = p.N;
        L.div_c = make_div_magic((uint32_t)p.C);
        L.flags = p.flags; L.m_bits = p.m_bits; L.zp_m = p.zp_m; L.zp_h = p.zp_h;
        L.W = p.W; L.R = p.R; L.Wproj = p.Wproj; L.bx = p.bx; L.bh = p.bh; L.bp = p.bp; L.bln = p.bln; L.P = p.P; L.L = p.L;
        for (int g = 0; g < 4; ++g) { L.eff_x[g] = p.eff_x[g]; L.eff_h[g] = p.eff_h[g]; L.eff_c[g] = p.eff_c[g]; L.eff_ln[g] = p.eff_ln[g]; }
        L.eff_m = p.eff_m; L.eff_proj = p.eff_proj;
        L.h_off = h_off; L.c_off = c_off;
        h_off += p.O; c_off += p.C;
        if (l + 1 < n) {
            L.seq = (int8_t *)dalloc((size_t)max_T * s->max_B * p.O);
            if (!L.seq) return fail(QLSTM_ERR_NOMEM);
        }
        L.m = (int8_t *)dalloc((size_t)s->max_B * p.C);
        L.part = (long long *)dalloc((size_t)sm_count * 2 * s->max_B * 8 * sizeof(long long));
        if (!L.m || !L.part) return fail(QLSTM_ERR_NOMEM);
        for (int plan = 0; plan < 2; ++plan) {
            const int per = plan == 0 ? sm_count / n : sm_count;
            L.cta0 = plan == 0 ? l * per : 0;
            L.n_cta = per;
            L.cpc = (p.C + per - 1) / per;
            L.rpc = (p.O + per - 1) / per;
            s->plan[plan].push_back(L);
            s->max_npc = std::max(s->max_npc, L.cpc * p.G);
        }
        s->max_I = std::max(s->max_I, p.I);
        s->max_O = std::max(s->max_O, p.O);
        if (p.flags & F_PROJECTION) s->max_C_proj = std::max(s->max_C_proj, p.C);
    }
    // the largest batch whose buffers fit
    while (s->max_B >= 1 && sk_smem_bytes(*s, sk_rows(s->max_B)) > (size_t)max_smem) s->max_B = sk_rows(s->max_B) / 2;
    if (s->max_B < 1) return fail(QLSTM_OK);
    s->smem = sk_smem_bytes(*s, sk_rows(s->max_B));
    s->cnt_words = (size_t)n * CNT_PER_LAYER + 16;
    s->cnt = (unsigned *)dalloc(2 * s->cnt_words * sizeof(unsigned));
    if (!s->cnt) return fail(QLSTM_ERR_NOMEM);
    if (cudaMemset(s->cnt, 0, 2 * s->cnt_words * sizeof(unsigned)) != cudaSuccess) return fail(QLSTM_ERR_CUDA);
    for (int plan = 0; plan < 2; ++plan) {
        s->plan_dev[plan] = (SkLayer *)dalloc(sizeof(SkLayer) * n);
        if (!s->plan_dev[plan]) return fail(QLSTM_ERR_NOMEM);
        if (cudaMemcpy(s->plan_dev[plan], s->plan[plan].data(), sizeof(SkLayer) * n, cudaMemcpyHostToDevice) != cudaSuccess)
            return fail(QLSTM_ERR_CUDA);
    }
    for (int NB : {1, 2, 4, 8, 16}) {
        if (NB > sk_rows(s->max_B)) break;
        if (cudaFuncSetAttribute(sk_kernel(NB), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s->smem) != cudaSuccess) return fail(QLSTM_OK);
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sk_kernel(NB), SK_THREADS, s->smem) != cudaSuccess || per_sm < 1)
            return fail(QLSTM_OK);
    }
    s->ok = true;
    *out = s;
    return QLSTM_OK;
}

bool stack_small_supported(const StackSmall *s, int T, int B) { return s && s->ok && B >= 1 && B <= s->max_B && T >= 1 && T <= s->max_T; }

// Where the whole-stack kernel is the faster path (measured, us per time step of the whole stack, this kernel against
// layer after layer): the wavefront's step costs one layer-step whatever the depth, the per-layer kernels' cost grows
// with it.  Eight 2048-cell layers: 26 / 127 at batch 1, 59 / 157 at 8, 107 / 158 at 16; five 1024-cell layers: 17 / 32
// at batch 4, 23 / 39 at 8, 33 / 39 at 16; two 256-cell layers: 6 / 10 at batch 2, 8.5 / 11 at 8; a single 2048-cell
// layer (nothing to overlap): 27 / 28 at batch 4, 39 / 27 at 8, 54 / 27 at 16.
bool stack_small_preferred(const StackSmall *s, int T, int B)
{
    if (!stack_small_supported(s, T, B)) return false;
    if (B <= 4) return true;
    // a call of one or two steps is launch- and barrier-bound layer by layer (33 against 54 us for one step of two
    // 256-cell layers at 8 rows)
    if (B <= 8 && (s->n_layers >= 2 || T <= 2)) return true;
    // 9 to 16 rows: measured for five and eight layers only, and only where the wavefront has steps to overlap (one
    // step per call at 16 rows: 448 against 375 us for the eight layers, 139 against 167 for the five)
    return s->n_layers >= 4 && T >= s->n_layers;
}

void stack_small_debug_timeout(StackSmall *s, unsigned missing_arrivals, unsigned long long limit_ns)
{
    if (!s) return;
    s->dbg_missing = missing_arrivals;
    s->dbg_limit_ns = missing_arrivals ? limit_ns : 0;
}

int stack_small_groups(const StackSmall *s, int *blocks_per_layer)
{
    if (!s || !s->ok) return 0;
    if (blocks_per_layer) *blocks_per_layer = s->plan[0].empty() ? 0 : s->plan[0][0].n_cta;
    return s->n_layers;
}

// schedule: 0 automatic (sequential for calls of a few steps, where a wavefront has nothing to overlap), 1 wavefront,
// 2 sequential
int launch_stack_small(StackSmall *s, const int8_t *x, int T, int B, int8_t *h, int16_t *c, int8_t *y, int *status,
                       int schedule, cudaStream_t st)
{
    SkCall k;
    memset(&k, 0, sizeof(k));
    k.T = T; k.B = B; k.n_layers = s->n_layers;
    k.x = x; k.h = h; k.c = c; k.y = y;
    unsigned *set = s->cnt + (size_t)(s->calls & 1u) * s->cnt_words;
    k.cnt = set;
    k.abort_word = set + (size_t)s->n_layers * CNT_PER_LAYER;
    k.cnt_next = s->cnt + (size_t)((s->calls + 1u) & 1u) * s->cnt_words;
    k.cnt_words = (int)s->cnt_words;
    ++s->calls;
    k.status = status;
    k.wait_limit_ns = s->dbg_limit_ns ? s->dbg_limit_ns : SK_WAIT_LIMIT_NS;
    k.missing_arrivals = s->dbg_missing;
    // a wavefront of L layers needs about L steps to fill; below that the layers are better run one after the other
    k.sequential = schedule == 2 || (schedule == 0 && (s->n_layers == 1 || T < s->n_layers)) ? 1 : 0;
    k.max_I = s->max_I; k.max_O = s->max_O; k.max_C_proj = s->max_C_proj; k.max_npc = s->max_npc;
    const SkLayer *layers = s->plan_dev[k.sequential];
    void *args[] = {(void *)&layers, (void *)&k};
    cudaError_t e = cudaLaunchCooperativeKernel(sk_kernel(sk_rows(B)), dim3(s->grid), dim3(SK_THREADS), args, s->smem, st);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return e == cudaErrorCooperativeLaunchTooLarge ? QLSTM_ERR_LAUNCH : QLSTM_ERR_CUDA;
    }
    return QLSTM_OK;
}

}  // namespace ql
