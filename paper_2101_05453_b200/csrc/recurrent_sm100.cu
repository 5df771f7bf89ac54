// Persistent recurrent kernel: all T steps of one LSTM layer in one cooperative launch.
//
// A block owns a range of cells for the whole sequence: its rows of R stay in shared memory.  Per step:
//
//   A  recurrent matmul   the block streams h^{t-1} (int8 [B][O]) through a TMA ring and runs tcgen05.mma kind::i8
//                         with the batch as M and its gate rows as N (dp4a mat-vecs at small batch).  Epilogue: + folded
//                         bias (saturating), rescale to the gate format, + the input projection X_t (+ the peephole
//                         terms on c^{t-1}) -> gate sums.
//   B  elementwise        integer layer norm, integer sigmoid / tanh, CIFG coupling, cell update, output-gate peephole
//                         on c^t, hidden state requantised to int8.
//        without layer norm: same block, same cells, straight after the epilogue - the gate sums never leave shared
//                         memory and there is no barrier between A and B.
//        with layer norm:  the statistics need every cell of a row (Section 3.2.6), so the gate sums go to L2 (one
//                         tensor-map store per block), a grid barrier follows, and phase B is partitioned as a flat
//                         range of the B x C cell grid (whole rows when layer norm and peephole combine: the output
//                         gate's statistics need c^t of the whole row).  (Keeping the cells with their block and adding
//                         per-row partial sums with atomics to totals in L2 was measured: 148 blocks adding to the same
//                         addresses cost more than the round trip they save - 49.5 against 37.4 us per step.)
//      -- grid barrier: the projection (or the next step's matmul) needs every m --
//   C  projection         partitioned by (batch tile, output slice); W_proj slice resident in shared memory,
//                         m^t streamed through the same TMA ring; epilogue requantises to int8 h^t.
//      -- grid barrier --
//
// Only the data that crosses blocks (h, m, and with layer norm the gate sums) goes through L2; the weights never move
// after the prologue.
//
// Every wait is bounded.  A wait that runs out sets the abort word; all CTAs observe it at the next
// barrier, leave the time loop together, free their tensor memory and return; the host reports
// QLSTM_ERR_TIMEOUT and the context stays usable.
#include <cstring>

#include "../../include/qlstm.h"
#include "../../include/qlstm_debug.h"
#include "act_table.cuh"
#include "fast_kernels.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace ql {

namespace {

constexpr int RTHREADS = 640;                 // warp 0 TMA producer, warp 1 MMA issuer, warps 2..9 matmul epilogues;
                                              // all 20 warps share the elementwise phase
constexpr int MAX_LN_ROWS = 4;                // flat elementwise phase: rows whose layer-norm statistics are held at once
constexpr int KB_BYTES = 128 * 128;           // one k-block of the A operand: 128 rows x 128 bytes
constexpr int STAGE_KB = 2;                   // k-blocks per ring stage: one bulk copy brings up to 32 KB
constexpr int STAGE_BYTES = STAGE_KB * KB_BYTES;
constexpr int MAX_STAGES = 4;
constexpr int SMALL_BATCH_MAX = 16;           // the dp4a mat-vec path exists up to this batch; the default crossover is lower
constexpr unsigned long long SPIN_LIMIT_NS = 2000000000ull;   // 2 s per grid barrier

// How one matmul phase uses the ring: owner o of n_own (one MMA issuer each) owns the stages o, o + n_own, ...
// (cnt[o] of them) and consumes n_chunks[o] chunks; uses[s]: times stage s is filled in the phase.
struct RingPlan {
    int n_own, n_max;
    int n_chunks[4], cnt[4];
    int uses[MAX_STAGES];
};

struct RecParams {
    int T, B, MT, Bpad;
    size_t h_stride;              // bytes between the two h operand buffers
    int C, O, G, N;
    uint32_t flags;
    int m_bits, zp_m, zp_h;
    int cpc, n_cta_a, nc_pad;
    int pn, npn, n_ptiles;
    int kb_h, kb_c, stages;
    int n_issue_c;                // projection: MMA issuers (= partial accumulators) sharing the K range
    RingPlan plan_a, plan_c;      // ring use of the recurrent matmul and of the projection
    int items_per_cta;            // layer norm: cells of the B x C grid per CTA in the flat elementwise phase
    int small;                    // small batch: dp4a mat-vec with warp reductions instead of TMA + tcgen05
    int npc;                      // gate rows per CTA = columns of its X box
    int x_rows;                   // rows of the X box: MT * 128 (B at small batch)
    uint32_t x_bytes;             // bytes of one X box: x_rows x npc int16
    uint32_t ho_bytes;            // peephole: bytes of the output gate's recurrent terms, x_rows x cpc int16
    uint32_t acc_off;             // byte offset in the ring (idle between the matmul phases) of the small-batch accumulators
    uint32_t row_bytes;           // layer norm + peephole: bytes of the row buffer of the elementwise phase
    int rpc;                      // small batch: projection rows per CTA
    const int8_t *R, *Wproj;      // packed weights (small-batch prologue copies its slices with plain loads)
    int fast_rescale_ok;          // every rescale of this layer has shift <= 0
    const int16_t *X;             // [T][B][N]
    int16_t *c;                   // [B][C]
    int8_t *y;                    // [T][B][O]
    int8_t *hbuf, *mbuf;
    int32_t *pre;                 // layer norm: gate sums [B][N] between the matmul and elementwise phases (int16 values,
                                  // or int32 X + H when a peephole term is still to be added)
    unsigned *bar;
    int *status;
    const int32_t *bh, *bp, *bln;
    const int16_t *P, *L;
    Scale eff_h[4], eff_c[4], eff_ln[4], eff_m, eff_proj;
    FastScale f_h[4], f_c[4], f_ln[4], f_m, f_proj;
    int gate_slot[4];             // canonical gate -> slot, -1 if absent
    unsigned long long spin_limit_ns;   // bound of one grid-barrier wait
    unsigned barrier_extra;             // 0; a test sets it to make the barrier wait for an arrival that never comes
    DivMagic div_c;               // division by C (layer-norm statistics) as a multiplication
    const uint8_t *tab;           // memoised sigmoid / tanh tables of this layer (act_table.cuh), copied into the idle ring
    ActTabLayout tab_lay;         // before every elementwise phase; used by the instantiations with TAB only
    unsigned long long *phase_ns; // null, or 6 accumulators: work and barrier wait of phases A, B, C (CTA 0)
};

struct RecCtl {
    uint64_t full[MAX_STAGES], empty[MAX_STAGES], acc_full[3], w_full, x_full, tab_full;
    uint32_t tmem_base;
    uint32_t rounds[MAX_STAGES];
    int abort_flag;
    long long red_sum[RTHREADS / 32][4], red_sq[RTHREADS / 32][4];
    LnRow ln_rows[MAX_LN_ROWS][4];
};

__device__ __forceinline__ bool wait_or_abort(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    // each attempt parks the thread for up to 20 us; 100 000 attempts bound the wait to about 2 s
    for (uint32_t i = 0; i < 100000u; ++i) {
        if (ptx::mbar_try_wait_parked(bar, parity, 20000u)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

__device__ __forceinline__ unsigned ld_acquire(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long globaltimer()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)::"memory");      // not to be moved across barriers
    return t;
}
// orders this thread's generic-proxy accesses to global memory with async-proxy (bulk copy) accesses to it
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }

// Grid-wide barrier on a monotonic counter: every thread's earlier global writes are ordered before the
// CTA barrier, one thread then publishes them with a release-add and polls with acquire loads.  Where the
// phase before it wrote data that other CTAs fetch with bulk copies (async proxy: the operands h and m),
// each writer first orders its generic-proxy writes against that proxy; the thread that issues the copies
// fences again on its side after the barrier.  Gate sums are read with ordinary loads and need neither.
// (Spreading the arrivals over several counters was tried: polling four words costs more than the serial
// tail of 148 atomics on one word.)
constexpr size_t BAR_BYTES = 64;                  // [0] counter, [1] abort word

__device__ __forceinline__ void grid_sync(const RecParams &p, unsigned &epoch, volatile int *abort_flag, bool wrote_operands)
{
    if (wrote_operands) fence_proxy_async_global();
    ptx::cta_sync();
    if (threadIdx.x == 0) {
        ++epoch;
        const unsigned target = epoch * gridDim.x + p.barrier_extra;
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.bar) : "memory");
        const unsigned long long t0 = globaltimer();
        unsigned spins = 0;
        while (ld_acquire(p.bar) < target) {
            if ((++spins & 63u) == 0u) {
                if (ld_acquire(p.bar + 1) != 0u) { *abort_flag = 1; break; }
                if (globaltimer() - t0 > p.spin_limit_ns) {
                    atomicExch(p.bar + 1, 1u);
                    *abort_flag = 1;
                    break;
                }
            }
        }
        if (*abort_flag) atomicExch(p.bar + 1, 1u);
    }
    ptx::cta_sync();
}

// FS: every scale of the layer shifts right (the usual case; decided per launch), so the rescale is the multiply-add
// form alone.  Otherwise each use chooses, and the form with a left shift is an out-of-line call: a call in an unrolled
// loop keeps the scheduler from interleaving the loop's independent chains (5 % of the step time at batch 256).
template <bool FS>
__device__ __forceinline__ int32_t rescale_sel(int32_t x, const Scale &s, const FastScale &f, int fast_ok)
{
    if constexpr (FS) return fast_rescale(x, f);
    else return fast_ok ? fast_rescale(x, f) : mbqm_cold(x, s);
}
template <bool FS>
__device__ __forceinline__ int32_t rescale_any(int32_t x, const Scale &s, const FastScale &f)
{
    if constexpr (FS) return fast_rescale(x, f);
    else return s.shift <= 0 ? fast_rescale(x, f) : mbqm_cold(x, s);
}
template <bool FS>
__device__ __forceinline__ int32_t ln_apply_sel(int32_t q, const LnRow &r, int32_t L, int32_t b, const Scale &eff, const FastScale &f)
{
    if constexpr (FS) return ln_apply_noshift(q, r, L, b, f);
    else return ln_apply_fast(q, r, L, b, eff, f);
}

// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ int32_t add_sat(int32_t a, int32_t b)
{
    int32_t d;
    asm("add.sat.s32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ int32_t lo16(uint32_t w) { return (int32_t)(w << 16) >> 16; }
__device__ __forceinline__ int32_t hi16(uint32_t w) { return (int32_t)w >> 16; }
__device__ __forceinline__ uint32_t pack16(int32_t lo, int32_t hi) { return ((uint32_t)lo & 0xffffu) | ((uint32_t)hi << 16); }

// Streamed matmul operands (h, m) live in global memory already in the shared-memory image the MMA reads:
// 128-row x 128-byte k-blocks, [row tile][k-block][row][128 B], 16-byte chunks swizzled by (row mod 8) as
// the 128-byte swizzle mode does.  A k-block (or a run of them) is then one contiguous bulk copy, which
// streams about twice as fast per SM as a tiled tensor-map box of 128 separate 128-byte rows.
__host__ __device__ __forceinline__ size_t tile_off(int row, int k, int nkb)
{
    return ((size_t)(row >> 7) * nkb + (k >> 7)) * KB_BYTES + (size_t)((row & 127) << 7) +
           (size_t)(((((k >> 4) & 7) ^ (row & 7)) << 4) | (k & 15));
}
// byte offset of element (row, k) of a [rows][K] operand: plain rows at small batch, tiled otherwise
__device__ __forceinline__ size_t operand_off(const RecParams &p, int row, int k, int K, int nkb)
{
    return p.small ? (size_t)row * K + k : tile_off(row, k, nkb);
}

// Views of what a block keeps in shared memory for its own cells (columns n = cell * G + slot of its gate rows).
struct OwnCells {
    int16_t *x_s;          // [x_rows][npc]   X_t, replaced in place by the gate sums
    int16_t *ho_s;         // [x_rows][cpc]   peephole only: the output gate's recurrent term H_o (its X stays in x_s)
    const int32_t *bh_s;   // [nc_pad]        folded bias of the recurrent accumulator
    const int16_t *P_s;    // [nc_pad]        peephole weights (0 where a gate has none)
    int u0;                // first cell
    int cells;             // cells owned (even; fewer than cpc in the last block)
};

// Matmul epilogue for one batch row b and the 8-column groups [g_begin, g_end) of this block's gate sums
// (Section 3.2.4 / 3.2.5).  Per column:
//   H   = sat16(rescale(sat32(acc + bh), eff_h))
//   out = sat16(X + H [+ sat16(rescale(P c^{t-1}, eff_c)) for the input and forget gates])
// X_t is in shared memory and is replaced in place.  Without layer norm a peephole layer finishes the input and forget
// gates here; the output gate waits for c^t: its X stays where it is and H goes to ho_s.  With layer norm and peephole
// (LN && PEEP) nothing can be finished yet: X + H goes to global memory as int32 and the elementwise phase adds the
// peephole terms row by row.
// TM: accumulators come from tensor memory (taddr; warp-collective loads, so every lane runs the loop) or from
// acc_row (int32, shared memory).  With three gates the groups are taken three at a time (24 columns = 8 cells), so
// that the slot of every column is a compile-time constant; g_begin is then a multiple of 3.
template <int G, bool LN, bool PEEP, bool TM, bool FS>
__device__ __forceinline__ void gate_sums_row(const RecParams &p, const OwnCells &oc, uint32_t taddr, const int32_t *acc_row,
                                              int b, int n0, int g_begin, int g_end, const int16_t *c_row, bool row_valid)
{
    constexpr int NB = (G == 4) ? 2 : 3;                     // groups per trip of the loop
    constexpr int NL = (G == 4) ? 2 : 1;                     // groups whose accumulators are loaded at once
    constexpr int SF = (G == 4) ? 1 : 0, SZ = SF + 1, SO = SF + 2;
    int16_t *xrow = oc.x_s + (size_t)b * p.npc;
#pragma unroll 1
    for (int gbase = g_begin; gbase < g_end; gbase += NB) {
        uint32_t r[NL][8];
        auto load_acc = [&](int first) {                     // accumulators of the groups first .. first + NL - 1 of this trip
            if (TM) {
                __syncwarp();                                // the TMEM loads are warp-collective
#pragma unroll
                for (int i = 0; i < NL; ++i)
                    if (gbase + first + i < g_end) ptx::tmem_ld_32x8(taddr + (uint32_t)((gbase + first + i) * 8), r[i]);   // warp-uniform
                ptx::tmem_ld_wait();
            } else {
#pragma unroll
                for (int i = 0; i < NL; ++i)
                    if (gbase + first + i < g_end) {
                        const int4 a0 = *reinterpret_cast<const int4 *>(acc_row + (gbase + first + i) * 8);
                        const int4 a1 = *reinterpret_cast<const int4 *>(acc_row + (gbase + first + i) * 8 + 4);
                        r[i][0] = a0.x; r[i][1] = a0.y; r[i][2] = a0.z; r[i][3] = a0.w;
                        r[i][4] = a1.x; r[i][5] = a1.y; r[i][6] = a1.z; r[i][7] = a1.w;
                    }
            }
        };
        if (NL == NB) {
            load_acc(0);
            if (TM && !row_valid) continue;
        }
        // c^{t-1} of the cells these columns belong to (peephole): 4 cells with four gates, 8 with three
        const int cell0 = (gbase * 8) / G;
        int32_t c_old[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (PEEP && !LN) {
            constexpr int NC = (G == 4) ? 4 : 8;
#pragma unroll
            for (int k = 0; k < NC; k += 2) {
                if (row_valid && cell0 + k < oc.cells) {
                    const uint32_t w = *reinterpret_cast<const uint32_t *>(c_row + cell0 + k);
                    c_old[k] = lo16(w); c_old[k + 1] = hi16(w);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            const int grp = gbase + i;
            if (grp >= g_end) break;
            if (NL != NB) {
                load_acc(i);
                if (TM && !row_valid) continue;
            }
            const int c8 = grp * 8;
            const uint4 x4 = *reinterpret_cast<const uint4 *>(xrow + c8);
            const uint32_t xw[4] = {x4.x, x4.y, x4.z, x4.w};
            const int4 b0 = *reinterpret_cast<const int4 *>(oc.bh_s + c8), b1 = *reinterpret_cast<const int4 *>(oc.bh_s + c8 + 4);
            const int32_t bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
            uint32_t pw[4] = {0, 0, 0, 0};
            if (PEEP && !LN) {
                const uint4 p4 = *reinterpret_cast<const uint4 *>(oc.P_s + c8);
                pw[0] = p4.x; pw[1] = p4.y; pw[2] = p4.z; pw[3] = p4.w;
            }
            int32_t o[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int col = i * 8 + j;                           // column inside this batch of groups
                const int gi = (G == 4) ? (j & 3) : col % 3;         // compile-time: gbase * 8 is a multiple of G
                const int cl = col / G;                              // cell inside this batch of groups
                const int32_t acc = add_sat((int32_t)r[NL == NB ? i : 0][j], bb[j]);
                const int32_t H = sat16(rescale_sel<FS>(acc, p.eff_h[gi], p.f_h[gi], p.fast_rescale_ok));
                const int32_t X = (j & 1) ? hi16(xw[j >> 1]) : lo16(xw[j >> 1]);
                if (LN) {
                    o[j] = X + H;                                    // saturated when packed (no peephole), or int32 as it is
                } else if (PEEP && gi == SO) {
                    o[j] = X;                                        // finished in phase B, once c^t exists
                    oc.ho_s[(size_t)b * p.cpc + cell0 + cl] = (int16_t)H;
                } else {
                    int32_t v = X + H;
                    if (PEEP && gi != SZ) {
                        const int32_t P = (j & 1) ? hi16(pw[j >> 1]) : lo16(pw[j >> 1]);
                        v += sat16(rescale_any<FS>(P * c_old[cl], p.eff_c[gi], p.f_c[gi]));
                    }
                    o[j] = v;                                        // saturated when packed
                }
            }
            if (LN && PEEP) {
                int32_t *dst = p.pre + (size_t)b * p.N + n0 + c8;
                *reinterpret_cast<int4 *>(dst) = make_int4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<int4 *>(dst + 4) = make_int4(o[4], o[5], o[6], o[7]);
                continue;
            }
            *reinterpret_cast<uint4 *>(xrow + c8) = make_uint4(ptx::pack_sat_s16(o[0], o[1]), ptx::pack_sat_s16(o[2], o[3]),
                                                               ptx::pack_sat_s16(o[4], o[5]), ptx::pack_sat_s16(o[6], o[7]));
        }
    }
}

// Phase C epilogue for one thread = one batch row and the columns [c_begin, c_end) of the projection tile, four at
// a time: sum of the issuers' partial accumulators + folded bias (saturating) -> rescale -> + zp_h -> int8.
template <bool FS>
__device__ __forceinline__ void phase_c_row(const RecParams &p, uint32_t taddr, int n_acc, int b, int t, int p0, int c_begin,
                                            int c_end, int8_t *h_next, bool row_valid)
{
    for (int col = c_begin; col < c_end; col += 4) {
        uint32_t r[4][4];
        __syncwarp();                                        // the TMEM loads are warp-collective
#pragma unroll
        for (int a = 0; a < 4; ++a)
            if (a < n_acc) ptx::tmem_ld_32x4(taddr + (uint32_t)(a * p.pn + col), r[a]);   // warp-uniform
        ptx::tmem_ld_wait();
        if (!row_valid || p0 + col >= p.O) continue;         // O is a multiple of 16: a group of 4 is inside or outside
        const int4 bias = __ldg(reinterpret_cast<const int4 *>(p.bp + p0 + col));
        const int32_t bb[4] = {bias.x, bias.y, bias.z, bias.w};
        uint32_t w = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int32_t sum = (int32_t)r[0][j];
#pragma unroll
            for (int a = 1; a < 4; ++a)
                if (a < n_acc) sum += (int32_t)r[a][j];      // partial sums of the other issuers (exact in int32)
            const int32_t acc = add_sat(sum, bb[j]);
            const int32_t hq = sat8(rescale_sel<FS>(acc, p.eff_proj, p.f_proj, p.fast_rescale_ok) + p.zp_h);
            w |= (uint32_t)(hq & 0xff) << (8 * j);
        }
        *reinterpret_cast<uint32_t *>(h_next + tile_off(b, p0 + col, p.kb_h)) = w;
        *reinterpret_cast<uint32_t *>(p.y + ((size_t)t * p.B + b) * p.O + p0 + col) = w;
    }
}

// ------------------------------------------------------------------------------------------------
// Phase B without layer norm: everything after the gate sums, for the block's own cells, two adjacent cells per task.

// G int16 values of two adjacent cells (cell index even): v[k][gi].  SRC: 0 shared memory (or data only this block
// writes), 1 read-only global data, 2 global data written by other blocks this step (L2 loads)
template <int G, int SRC>
__device__ __forceinline__ void load_pair_i16(const int16_t *ptr, int32_t (&v)[2][4])
{
    if (G == 4) {
        const uint4 *q4 = reinterpret_cast<const uint4 *>(ptr);
        const uint4 q = SRC == 0 ? *q4 : (SRC == 1 ? __ldg(q4) : __ldcg(q4));
        v[0][0] = lo16(q.x); v[0][1] = hi16(q.x); v[0][2] = lo16(q.y); v[0][3] = hi16(q.y);
        v[1][0] = lo16(q.z); v[1][1] = hi16(q.z); v[1][2] = lo16(q.w); v[1][3] = hi16(q.w);
    } else {
        const uint32_t *w = reinterpret_cast<const uint32_t *>(ptr);
        uint32_t a, b, c;
        if (SRC == 0) { a = w[0]; b = w[1]; c = w[2]; }
        else if (SRC == 1) { a = __ldg(w); b = __ldg(w + 1); c = __ldg(w + 2); }
        else { a = __ldcg(w); b = __ldcg(w + 1); c = __ldcg(w + 2); }
        v[0][0] = lo16(a); v[0][1] = hi16(a); v[0][2] = lo16(b);
        v[1][0] = hi16(b); v[1][1] = lo16(c); v[1][2] = hi16(c);
        v[0][3] = 0; v[1][3] = 0;
    }
}
// The same pair from global data written by other blocks this step, as loaded (so that several loads can be in flight
// before the first is unpacked), and its unpacking.
template <int G>
__device__ __forceinline__ uint4 load_pair_raw(const int16_t *ptr)
{
    if (G == 4) return __ldcg(reinterpret_cast<const uint4 *>(ptr));
    const uint32_t *w = reinterpret_cast<const uint32_t *>(ptr);
    return make_uint4(__ldcg(w), __ldcg(w + 1), __ldcg(w + 2), 0u);
}
template <int G>
__device__ __forceinline__ void unpack_pair(const uint4 &q, int32_t (&v)[2][4])
{
    if (G == 4) {
        v[0][0] = lo16(q.x); v[0][1] = hi16(q.x); v[0][2] = lo16(q.y); v[0][3] = hi16(q.y);
        v[1][0] = lo16(q.z); v[1][1] = hi16(q.z); v[1][2] = lo16(q.w); v[1][3] = hi16(q.w);
    } else {
        v[0][0] = lo16(q.x); v[0][1] = hi16(q.x); v[0][2] = lo16(q.y);
        v[1][0] = hi16(q.y); v[1][1] = lo16(q.z); v[1][2] = hi16(q.z);
        v[0][3] = 0; v[1][3] = 0;
    }
}

template <int G>
__device__ __forceinline__ void load_pair_i32(const int32_t *ptr, int32_t (&v)[2][4])      // read-only global data
{
#pragma unroll
    for (int k = 0; k < 2; ++k)
#pragma unroll
        for (int g = 0; g < 4; ++g) v[k][g] = g < G ? __ldg(ptr + k * G + g) : 0;
}

__device__ __forceinline__ void store_hidden_pair(const RecParams &p, int b, int u, int t, int32_t m0, int32_t m1, int8_t *h_next)
{
    const uint16_t v = (uint16_t)((m0 & 0xff) | ((m1 & 0xff) << 8));
    if (p.flags & F_PROJECTION) {
        *reinterpret_cast<uint16_t *>(p.mbuf + operand_off(p, b, u, p.C, p.kb_c)) = v;
    } else {
        *reinterpret_cast<uint16_t *>(h_next + operand_off(p, b, u, p.O, p.kb_h)) = v;
        *reinterpret_cast<uint16_t *>(p.y + ((size_t)t * p.B + b) * p.O + u) = v;
    }
}

// The nonlinearities of the elementwise phase: the fixed-point definition, or its memoised values (TAB).
template <bool TAB>
__device__ __forceinline__ int32_t gate_sigmoid(const ActTabs &at, int32_t x)
{
    if constexpr (TAB) return tab_sigmoid(at, x);
    else return sigmoid_q_fast(x, 3);
}
template <bool TAB>
__device__ __forceinline__ int32_t gate_tanh(const ActTabs &at, int32_t x)
{
    if constexpr (TAB) return tab_tanh_gate(at, x);
    else return tanh_q_fast(x, 3);
}
template <bool TAB, bool FS>
__device__ __forceinline__ int32_t hidden_of(const RecParams &p, const ActTabs &at, int32_t o, int32_t c_new)
{
    int32_t tc;
    if constexpr (TAB) tc = tab_tanh_cell(at, c_new);
    else tc = tanh_q_fast(c_new, p.m_bits);
    return sat8(rescale_any<FS>(o * tc, p.eff_m, p.f_m) + p.zp_m);                      // Section 3.2.7
}

// One pair of the block's own cells (local pair k of row b), gate sums in shared memory.
template <int G, bool PEEP, bool TAB, bool FS>
__device__ __forceinline__ void own_cell_pair(const RecParams &p, const OwnCells &oc, const ActTabs &at, int b, int k, int t,
                                              int8_t *h_next)
{
    constexpr int SI = 0, SF = (G == 4) ? 1 : 0, SZ = SF + 1, SO = SF + 2;
    const int ul = 2 * k, nl = ul * G;                     // local cell and column
    const int u = oc.u0 + ul;
    int16_t *c_ptr = p.c + (size_t)b * p.C + u;
    int32_t a[2][4];
    load_pair_i16<G, 0>(oc.x_s + (size_t)b * p.npc + nl, a);
    const uint32_t cw = *reinterpret_cast<const uint32_t *>(c_ptr);
    const int32_t c_old[2] = {lo16(cw), hi16(cw)};
    int32_t c_new[2], m[2];
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const int32_t f = gate_sigmoid<TAB>(at, a[q][SF]), z = gate_tanh<TAB>(at, a[q][SZ]);
        int32_t i;
        if (G == 4) i = gate_sigmoid<TAB>(at, a[q][SI]);
        else { i = 32768 - f; if (i > 32767) i = 32767; }          // coupled input gate, Section 3.2.9
        c_new[q] = cell_update_fast(i, z, f, c_old[q], p.m_bits);
        int32_t ao = a[q][SO];
        if (PEEP) {
            const int32_t H = oc.ho_s[(size_t)b * p.cpc + ul + q], P = oc.P_s[nl + q * G + SO];
            ao = sat16(ao + H + sat16(rescale_any<FS>(P * c_new[q], p.eff_c[SO], p.f_c[SO])));   // Eq. 5: o sees c^t
        }
        m[q] = hidden_of<TAB, FS>(p, at, gate_sigmoid<TAB>(at, ao), c_new[q]);
    }
    *reinterpret_cast<uint32_t *>(c_ptr) = pack16(c_new[0], c_new[1]);
    store_hidden_pair(p, b, u, t, m[0], m[1], h_next);
}

// All (row, cell pair) tasks of the block, consecutive threads on consecutive pairs of a row: the gate sums of a row's
// pairs are contiguous in shared memory.
template <int G, bool PEEP, bool TAB, bool FS>
__device__ __forceinline__ void phase_b_own(const RecParams &p, const OwnCells &oc, const ActTabs &at, int t, int8_t *h_next)
{
    const int pairs = oc.cells >> 1, total = p.B * pairs;
    for (int i = threadIdx.x; i < total; i += RTHREADS) {
        const int b = i / pairs, k = i - b * pairs;
        own_cell_pair<G, PEEP, TAB, FS>(p, oc, at, b, k, t, h_next);
    }
}

// ------------------------------------------------------------------------------------------------
// Phase B with layer norm: elementwise work on a contiguous range of the B x C cell grid, gate sums from L2.

// Warp-level part of the statistics reduction: per-gate sum / sum of squares of this warp into shared memory.
// The warp-wide adds are the hardware's 32-bit integer reduction (one instruction per value, where a shuffle tree is
// ten per 64-bit value and the shuffle unit issues one per clock for the whole SM): a thread's sum of at most a row of
// int16 values fits 32 bits as it is; its sum of squares (below 2^44) goes as its low 20 bits and the rest.
template <int G>
__device__ __forceinline__ void warp_reduce_stats(RecCtl *ctl, const long long (&sum)[4], const long long (&sq)[4])
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const int a = __reduce_add_sync(0xffffffffu, (int)sum[g]);
        const unsigned long long q = (unsigned long long)sq[g];
        const unsigned lo = __reduce_add_sync(0xffffffffu, (unsigned)(q & 0xfffffu));
        const unsigned hi = __reduce_add_sync(0xffffffffu, (unsigned)(q >> 20));
        if (lane == 0) { ctl->red_sum[warp][g] = a; ctl->red_sq[warp][g] = (long long)(((unsigned long long)hi << 20) + lo); }
    }
}

// Block-wide reduction (all warps contribute to one row) into ctl->ln_rows[slot][*].
template <int G>
__device__ __forceinline__ void block_reduce_stats(RecCtl *ctl, const long long (&sum)[4], const long long (&sq)[4],
                                                   const DivMagic &div_n, int slot)
{
    warp_reduce_stats<G>(ctl, sum, sq);
    ptx::cta_sync();
    if (threadIdx.x < G) {
        long long a = 0, b = 0;
        for (int w = 0; w < RTHREADS / 32; ++w) { a += ctl->red_sum[w][threadIdx.x]; b += ctl->red_sq[w][threadIdx.x]; }
        ctl->ln_rows[slot][threadIdx.x] = make_ln_row(ln_stats_fast(a, b, div_n));
    }
    ptx::cta_sync();
}

template <int G>
__device__ __forceinline__ void load_pair_i32_cg(const int32_t *ptr, int32_t (&v)[2][4])   // written by other blocks this step
{
#pragma unroll
    for (int k = 0; k < 2; ++k)
#pragma unroll
        for (int g = 0; g < 4; ++g) v[k][g] = g < G ? __ldcg(ptr + k * G + g) : 0;
}

// Two adjacent cells (u even) of row b, every step after the gate sums (layer norm without peephole).
template <int G, bool LN, bool PEEP, bool TAB, bool FS>
__device__ __forceinline__ void flat_cell_pair(const RecParams &p, const ActTabs &at, const LnRow *lr, int b, int u, int t,
                                               int8_t *h_next)
{
    constexpr int SI = 0, SF = (G == 4) ? 1 : 0, SZ = SF + 1, SO = SF + 2;
    const size_t nb = (size_t)b * p.N + (size_t)u * G;
    const int nu = u * G;
    int16_t *c_ptr = p.c + (size_t)b * p.C + u;
    const uint32_t cw = *reinterpret_cast<const uint32_t *>(c_ptr);
    const int32_t c_old[2] = {lo16(cw), hi16(cw)};
    int32_t a[2][4], P[2][4];
    if (PEEP) {
        load_pair_i32_cg<G>(p.pre + nb, a);
        load_pair_i16<G, 1>(p.P + nu, P);
#pragma unroll
        for (int k = 0; k < 2; ++k)
#pragma unroll
            for (int g = 0; g < G; ++g) {
                if (g == SO) continue;
                int32_t v = a[k][g];
                if (g != SZ) v += sat16(rescale_any<FS>(P[k][g] * c_old[k], p.eff_c[g], p.f_c[g]));
                a[k][g] = sat16(v);
            }
    } else {
        load_pair_i16<G, 2>((const int16_t *)p.pre + nb, a);
        if (LN) {
            int32_t L[2][4], bl[2][4];
            load_pair_i16<G, 1>(p.L + nu, L);
            load_pair_i32<G>(p.bln + nu, bl);
#pragma unroll
            for (int k = 0; k < 2; ++k)
#pragma unroll
                for (int g = 0; g < G; ++g) a[k][g] = ln_apply_sel<FS>(a[k][g], lr[g], L[k][g], bl[k][g], p.eff_ln[g], p.f_ln[g]);
        }
    }
    int32_t c_new[2], m[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int32_t f = gate_sigmoid<TAB>(at, a[k][SF]), z = gate_tanh<TAB>(at, a[k][SZ]);
        int32_t i;
        if (G == 4) i = gate_sigmoid<TAB>(at, a[k][SI]);
        else { i = 32768 - f; if (i > 32767) i = 32767; }          // coupled input gate, Section 3.2.9
        c_new[k] = cell_update_fast(i, z, f, c_old[k], p.m_bits);
        int32_t ao = a[k][SO];
        if (PEEP) ao = sat16(ao + sat16(rescale_any<FS>(P[k][SO] * c_new[k], p.eff_c[SO], p.f_c[SO])));
        const int32_t o = gate_sigmoid<TAB>(at, ao);
        m[k] = hidden_of<TAB, FS>(p, at, o, c_new[k]);
    }
    *reinterpret_cast<uint32_t *>(c_ptr) = pack16(c_new[0], c_new[1]);
    store_hidden_pair(p, b, u, t, m[0], m[1], h_next);
}

template <int G, bool LN, bool PEEP, bool TAB, bool FS>
__device__ __forceinline__ void phase_b_flat(const RecParams &p, RecCtl *ctl, const ActTabs &at, int t, int8_t *h_next)
{
    const int total = p.B * p.C;
    const int i0 = blockIdx.x * p.items_per_cta;
    int i1 = i0 + p.items_per_cta;
    if (i1 > total) i1 = total;
    if (i0 >= i1) return;
    const int b_first = i0 / p.C, b_last = (i1 - 1) / p.C;
    for (int rb = b_first; rb <= b_last; rb += MAX_LN_ROWS) {
        const int re = (rb + MAX_LN_ROWS - 1 < b_last) ? rb + MAX_LN_ROWS - 1 : b_last;
        if (LN) {
            // statistics of all rows of this batch at once: the warps are split evenly over the rows
            const int nrows = re - rb + 1;
            const int wpr = (RTHREADS / 32) / nrows;                       // warps per row
            const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
            const int r = warp / wpr;
            long long sum[4] = {0, 0, 0, 0}, sq[4] = {0, 0, 0, 0};
            if (r < nrows) {
                const int16_t *row = (const int16_t *)p.pre + (size_t)(rb + r) * p.N;
                const int tig = (warp - r * wpr) * 32 + lane, gs = wpr * 32;
                // eight independent loads in flight per thread, kept packed until all are issued: the row comes from
                // L2, and every trip of this loop pays that latency once
                for (int u0 = 2 * tig; u0 < p.C; u0 += 16 * gs) {
                    uint4 raw[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const int u = u0 + 2 * gs * k;
                        raw[k] = u < p.C ? load_pair_raw<G>(row + (size_t)u * G) : make_uint4(0u, 0u, 0u, 0u);
                    }
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        int32_t v[2][4];
                        unpack_pair<G>(raw[k], v);
#pragma unroll
                        for (int g = 0; g < G; ++g) {
                            sum[g] += v[0][g] + v[1][g];
                            sq[g] += (long long)(v[0][g] * v[0][g]) + (long long)(v[1][g] * v[1][g]);
                        }
                    }
                }
            }
            warp_reduce_stats<G>(ctl, sum, sq);
            ptx::cta_sync();
            if (threadIdx.x < nrows * 4 && (threadIdx.x & 3) < G) {
                const int rr = threadIdx.x >> 2, g = threadIdx.x & 3;
                long long a = 0, b = 0;
                for (int w = rr * wpr; w < (rr + 1) * wpr; ++w) { a += ctl->red_sum[w][g]; b += ctl->red_sq[w][g]; }
                ctl->ln_rows[rr][g] = make_ln_row(ln_stats_fast(a, b, p.div_c));
            }
            ptx::cta_sync();
        }
        const int j0 = i0 > rb * p.C ? i0 : rb * p.C;
        const int j1 = i1 < (re + 1) * p.C ? i1 : (re + 1) * p.C;
        // (row, cell) of a thread's tasks: one division for the first, then steps of 2 RTHREADS cells
        constexpr int step = 2 * RTHREADS;
        const int sb = step / p.C, su = step - sb * p.C;
        int i = j0 + 2 * (int)threadIdx.x;
        int b = i / p.C, u = i - b * p.C;
        for (; i < j1; i += step) {
            flat_cell_pair<G, LN, PEEP, TAB, FS>(p, at, ctl->ln_rows[b - rb], b, u, t, h_next);
            b += sb; u += su;
            if (u >= p.C) { u -= p.C; ++b; }
        }
        if (LN) ptx::cta_sync();      // the statistics slots are reused by the next batch of rows
    }
}

// Layer norm with peephole: the gate sums need their peephole term before the statistics, and the output
// gate's statistics need c^t of the whole row, so a row is processed by one CTA in three passes.
template <int G, bool TAB, bool FS>
__device__ __forceinline__ void phase_b_ln_peep(const RecParams &p, RecCtl *ctl, const ActTabs &at, int t, int8_t *h_next,
                                                int16_t *row_s)
{
    constexpr int SI = 0, SF = (G == 4) ? 1 : 0, SZ = SF + 1, SO = SF + 2;
    const int rows_per_cta = p.items_per_cta / p.C;
    const int b0 = blockIdx.x * rows_per_cta;
    const int b1 = (b0 + rows_per_cta < p.B) ? b0 + rows_per_cta : p.B;
    int16_t *pre_s = row_s, *cnew_s = row_s + (size_t)p.C * G;
    for (int b = b0; b < b1; ++b) {
        int16_t *c_row = p.c + (size_t)b * p.C;
        const int32_t *xh = p.pre + (size_t)b * p.N;
        const LnRow *lr = ctl->ln_rows[0];
        long long sum[4] = {0, 0, 0, 0}, sq[4] = {0, 0, 0, 0};
        for (int u = threadIdx.x; u < p.C; u += RTHREADS) {
            const int32_t c_old = c_row[u];
#pragma unroll
            for (int g = 0; g < G; ++g) {
                if (g == SO) continue;
                const int n = u * G + g;
                int32_t v = xh[n];
                if (g != SZ) v += sat16(rescale_any<FS>((int32_t)__ldg(p.P + n) * c_old, p.eff_c[g], p.f_c[g]));
                v = sat16(v);
                pre_s[n] = (int16_t)v;
                sum[g] += v;
                sq[g] += (long long)(v * v);
            }
        }
        block_reduce_stats<G>(ctl, sum, sq, p.div_c, 0);
        long long sum_o[4] = {0, 0, 0, 0}, sq_o[4] = {0, 0, 0, 0};
        for (int u = threadIdx.x; u < p.C; u += RTHREADS) {
            const int nb = u * G;
            int32_t a[4];
#pragma unroll
            for (int g = 0; g < G; ++g)
                if (g != SO) a[g] = ln_apply_sel<FS>(pre_s[nb + g], lr[g], __ldg(p.L + nb + g), __ldg(p.bln + nb + g), p.eff_ln[g], p.f_ln[g]);
            const int32_t f = gate_sigmoid<TAB>(at, a[SF]), z = gate_tanh<TAB>(at, a[SZ]);
            int32_t i;
            if (G == 4) i = gate_sigmoid<TAB>(at, a[SI]);
            else { i = 32768 - f; if (i > 32767) i = 32767; }
            const int32_t c_new = cell_update_fast(i, z, f, c_row[u], p.m_bits);
            c_row[u] = (int16_t)c_new;
            cnew_s[u] = (int16_t)c_new;
            const int32_t v = sat16(xh[nb + SO] + sat16(rescale_any<FS>((int32_t)__ldg(p.P + nb + SO) * c_new, p.eff_c[SO], p.f_c[SO])));
            pre_s[nb + SO] = (int16_t)v;
            sum_o[SO] += v;
            sq_o[SO] += (long long)(v * v);
        }
        ptx::cta_sync();              // statistics of i, f, z are consumed; their slots are reused for o
        block_reduce_stats<G>(ctl, sum_o, sq_o, p.div_c, 0);
        for (int u = threadIdx.x; u < p.C; u += RTHREADS) {
            const int n = u * G + SO;
            const int32_t ao = ln_apply_sel<FS>(pre_s[n], lr[SO], __ldg(p.L + n), __ldg(p.bln + n), p.eff_ln[SO], p.f_ln[SO]);
            const int32_t o = gate_sigmoid<TAB>(at, ao);
            const int32_t m = hidden_of<TAB, FS>(p, at, o, cnew_s[u]);
            if (p.flags & F_PROJECTION) {
                p.mbuf[operand_off(p, b, u, p.C, p.kb_c)] = (int8_t)m;
            } else {
                h_next[operand_off(p, b, u, p.O, p.kb_h)] = (int8_t)m;
                p.y[((size_t)t * p.B + b) * p.O + u] = (int8_t)m;
            }
        }
        ptx::cta_sync();
    }
}

// ------------------------------------------------------------------------------------------------
// Small batch (default: B <= 4; measured crossover: from 8 rows on the tensor-core path is faster; selectable up to
// SMALL_BATCH_MAX = 16 rows):
// the matmuls are mat-vec products, far too small for a 128-row tensor-core tile
// and dominated by TMA / TMEM round-trip latency.  Each warp takes whole weight rows from shared memory,
// lanes split K in 128-byte strides (conflict-free), dp4a accumulates, one warp reduction per (row, batch).

__device__ __forceinline__ void stage_rows(int8_t *dst_s, const int8_t *src, int bytes)
{
    const uint4 *s4 = reinterpret_cast<const uint4 *>(src);
    uint4 *d4 = reinterpret_cast<uint4 *>(dst_s);
    for (int i = threadIdx.x; i < (bytes >> 4); i += RTHREADS) d4[i] = __ldcg(s4 + i);   // L2 loads: written by other CTAs this step
    ptx::cta_sync();
}

template <int BMAX>
__device__ __forceinline__ int32_t warp_dots(const int8_t *w_row, const int8_t *v_s, int K, int lane)
{
    const int32_t *rw = reinterpret_cast<const int32_t *>(w_row);
    int32_t part[BMAX];
#pragma unroll
    for (int b = 0; b < BMAX; ++b) part[b] = 0;
    for (int w = lane; w < (K >> 2); w += 32) {
        const int32_t r = rw[w];
#pragma unroll
        for (int b = 0; b < BMAX; ++b)
            part[b] = __dp4a(r, reinterpret_cast<const int32_t *>(v_s + (size_t)b * K)[w], part[b]);
    }
    int32_t mine = 0;
#pragma unroll
    for (int b = 0; b < BMAX; ++b) {
        const int32_t sum = __reduce_add_sync(0xffffffffu, part[b]);
        if (lane == b) mine = sum;
    }
    return mine;                                   // lane b holds the dot product with batch row b
}

// recurrent accumulators of the block's gate rows into shared memory, acc_s [B][nc_pad] int32
template <int BMAX>
__device__ __forceinline__ void phase_a_small(const RecParams &p, int cur, int n_cnt, const int8_t *R_s, int8_t *stage_s,
                                              int32_t *acc_s)
{
    stage_rows(stage_s, p.hbuf + (size_t)cur * p.h_stride, p.B * p.O);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int n = warp; n < n_cnt; n += RTHREADS / 32) {
        const int32_t mine = warp_dots<BMAX>(R_s + (size_t)n * p.O, stage_s, p.O, lane);
        if (lane < p.B) acc_s[lane * p.nc_pad + n] = mine;
    }
}

template <int BMAX>
__device__ __forceinline__ void phase_c_small(const RecParams &p, int t, int p_lo, int cnt, const int8_t *Wp_s,
                                              int8_t *stage_s, int8_t *h_next)
{
    stage_rows(stage_s, p.mbuf, p.B * p.C);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int r = warp; r < cnt; r += RTHREADS / 32) {
        const int32_t mine = warp_dots<BMAX>(Wp_s + (size_t)r * p.C, stage_s, p.C, lane);
        if (lane < p.B) {
            const int b = lane, o = p_lo + r;
            const int32_t acc = add_sat(mine, __ldg(p.bp + o));
            const int32_t hq = sat8(rescale_sel<false>(acc, p.eff_proj, p.f_proj, p.fast_rescale_ok) + p.zp_h);
            h_next[(size_t)b * p.O + o] = (int8_t)hq;
            p.y[((size_t)t * p.B + b) * p.O + o] = (int8_t)hq;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Operand ring of the tensor-core phases.  A chunk is up to STAGE_KB k-blocks, contiguous in the tiled global
// image.  One producer thread issues the bulk copies; several issuer threads, each with its own accumulator,
// consume them: a single thread's issue latency (wait, descriptors, 4 MMAs per k-block, commit), not the copy
// rate, is what bounds a one-issuer loop.
// Within a phase every stage belongs to exactly one issuer: owner o of n_own uses the stages o, o + n_own, ...
// in turn for its chunks.  A thread therefore only ever waits for the next round of a stage whose previous round
// it has consumed itself (an mbarrier parity wait cannot tell round r + 1 from round r - 1).  Between phases the
// CTA-wide barriers order everything, so a stage may change owner from one phase to the next.  rounds[s] counts
// the uses of stage s so far: the parity of a use is its round number mod 2.

struct Ring {
    uint8_t *base;
    volatile uint32_t *rounds;       // shared memory, advanced by one thread between phases
};

// Chunks of a phase: `contig`: owner o streams operand tile o, chunk j = k-blocks [j STAGE_KB, ...) of that tile;
// else all owners share one tile and owner o takes its chunks o, o + n_own, ...  kb_total: k-blocks per tile.
// The producer visits the owners round-robin, so that it only ever waits for a stage of the owner whose chunk
// is due.  No division in these single-thread loops: their latency is the pace of the whole phase.
__device__ __forceinline__ void ring_produce(RecCtl *ctl, const Ring &r, const RingPlan &pl, bool contig, int kb_total,
                                             const int8_t *src, volatile int *abort_flag)
{
    int kk[4] = {0, 0, 0, 0};
    uint32_t rr[4] = {0, 0, 0, 0};
    for (int j = 0; j < pl.n_max; ++j) {
#pragma unroll
        for (int o = 0; o < 4; ++o) {
            if (o >= pl.n_own || j >= pl.n_chunks[o]) continue;
            const int c = contig ? j : o + j * pl.n_own;          // chunk number inside the tile
            const uint32_t stage = (uint32_t)(o + pl.n_own * kk[o]);
            const uint32_t par = (r.rounds[stage] + rr[o]) & 1u;
            if (++kk[o] == pl.cnt[o]) { kk[o] = 0; ++rr[o]; }
            const int kb = c * STAGE_KB;
            const uint32_t bytes = (uint32_t)((kb_total - kb < STAGE_KB ? kb_total - kb : STAGE_KB) * KB_BYTES);
            if (!wait_or_abort(&ctl->empty[stage], par ^ 1u, abort_flag)) return;
            ptx::mbar_arrive_expect_tx(&ctl->full[stage], bytes);
            ptx::bulk_load_1d(r.base + (size_t)stage * STAGE_BYTES, src + ((size_t)(contig ? o : 0) * kb_total + kb) * KB_BYTES, bytes,
                              &ctl->full[stage]);
        }
    }
}

// issuer = owner `me`: all k-blocks of each of its chunks into accumulator d_tmem.
// b_base is the shared-memory address of the resident B operand, b_kb_bytes its bytes per k-block.
__device__ __forceinline__ bool ring_issue(RecCtl *ctl, const Ring &r, const RingPlan &pl, int me, bool contig, int kb_total,
                                           uint32_t b_base, uint32_t b_kb_bytes, uint32_t d_tmem, uint32_t idesc,
                                           volatile int *abort_flag)
{
    const uint64_t a_desc0 = ptx::smem_desc_k_sw128(ptx::smem_u32(r.base));
    const uint64_t b_desc0 = ptx::smem_desc_k_sw128(b_base);
    const int n_mine = pl.n_chunks[me], cnt = pl.cnt[me];
    int kk = 0;
    uint32_t rr = 0;
    bool acc = false;
    for (int j = 0; j < n_mine; ++j) {
        const uint32_t stage = (uint32_t)(me + pl.n_own * kk);
        const uint32_t par = (r.rounds[stage] + rr) & 1u;
        if (++kk == cnt) { kk = 0; ++rr; }
        if (!wait_or_abort(&ctl->full[stage], par, abort_flag)) return false;
        ptx::tc_fence_after();
        const int kb0 = (contig ? j : me + j * pl.n_own) * STAGE_KB;
        uint64_t a_desc = a_desc0 + (uint64_t)(stage * (STAGE_BYTES >> 4));
        uint64_t b_desc = b_desc0 + (uint64_t)(((uint32_t)kb0 * b_kb_bytes) >> 4);
        const int nk = kb_total - kb0 < STAGE_KB ? kb_total - kb0 : STAGE_KB;
        for (int k2 = 0; k2 < nk; ++k2) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                ptx::mma_i8_ss(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, acc);
                acc = true;
            }
            a_desc += KB_BYTES >> 4;
            b_desc += b_kb_bytes >> 4;
        }
        ptx::mma_commit(&ctl->empty[stage]);
    }
    return true;
}

// after a phase: advance the round counters by the uses of each stage in that phase
__device__ __forceinline__ void ring_advance(const Ring &r, const RingPlan &pl)
{
#pragma unroll
    for (int s = 0; s < MAX_STAGES; ++s) r.rounds[s] += (uint32_t)pl.uses[s];
}

// Abort path only, kept out of line so that it does not take part in the kernel's register allocation (inlined it cost
// the time loop 3 %): wait, bounded, until no tensor-map copy into the X box is still on its way.
__device__ __noinline__ void drain_box_requests(uint64_t *x_full)
{
    for (uint32_t par = 0; par < 2; ++par)
        for (int i = 0; i < 2000 && !ptx::mbar_try_wait_parked(x_full, par, 1000u); ++i) {}
}

// One instantiation per variant (gates, layer norm, peephole): each keeps only its own epilogue and elementwise code,
// which is what lets the register allocator fit them without spilling.
// MODE: 0 any scales, nonlinearities evaluated; 1 every scale shifts right (FS); 2 FS and the nonlinearities memoised (TAB)
template <int G, bool LN, bool PEEP, int MODE>
__global__ void __launch_bounds__(RTHREADS, 1)
k_recurrent_sm100(const __grid_constant__ CUtensorMap map_R, const __grid_constant__ CUtensorMap map_Wp,
                  const __grid_constant__ CUtensorMap map_X, const __grid_constant__ CUtensorMap map_pre, RecParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const bool proj = (p.flags & F_PROJECTION) != 0;
    constexpr bool ln = LN, peep = PEEP;
    constexpr bool TAB = MODE == 2, FS = MODE >= 1;
    // layout: [ring stages][R slice][Wproj slice][X box][H_o (peephole) | row buffer (layer norm + peephole)]
    //         [per-column constants][control]
    uint8_t *ring = smem;
    uint8_t *R_s = ring + (size_t)p.stages * STAGE_BYTES;
    // R slice: npc rows per k-block.  The MMA reads nc_pad (npc rounded up to 16) rows per k-block: the up to 8 extra
    // rows are the head of the next k-block (of the next region after the last one), and their columns are never read
    uint8_t *Wp_s = R_s + (size_t)p.kb_h * p.npc * 128;
    int16_t *x_s = (int16_t *)(Wp_s + (proj ? (size_t)p.kb_c * p.pn * 128 : 0));
    uint8_t *after_x = (uint8_t *)x_s + (((size_t)p.x_bytes + 1023) & ~(size_t)1023);
    int16_t *ho_s = (int16_t *)after_x;
    int16_t *row_s = (int16_t *)after_x;
    const size_t extra = (size_t)(ln ? p.row_bytes : p.ho_bytes);
    int32_t *bh_s = (int32_t *)(after_x + ((extra + 15) & ~(size_t)15));
    int16_t *P_s = (int16_t *)(bh_s + p.nc_pad);
    RecCtl *ctl = (RecCtl *)(P_s + p.nc_pad);
    // between the matmul phases the ring is idle: at small batch the staged operand and the accumulators live there
    int8_t *stage_s = (int8_t *)ring;                                           // small batch: staged h / m, [B][K]
    int32_t *acc_s = (int32_t *)(ring + p.acc_off);                             // small batch: [B][nc_pad]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cta = blockIdx.x;
    volatile int *abort_flag = &ctl->abort_flag;
    const bool has_cells = cta < p.n_cta_a;
    const bool has_ptile = proj && cta < p.n_ptiles;
    const int n0 = cta * p.cpc * G;
    int n_cnt = p.cpc * G;
    if (n0 + n_cnt > p.N) n_cnt = p.N - n0;
    if (!has_cells) n_cnt = 0;
    const int tile_mi = has_ptile ? cta / p.npn : 0, tile_p0 = has_ptile ? (cta % p.npn) * p.pn : 0;
    const uint32_t acc_cols_a = (uint32_t)(p.MT * p.nc_pad);
    uint32_t tmem_cols = 32;
    while (tmem_cols < acc_cols_a + (uint32_t)(proj ? p.pn * p.n_issue_c : 0)) tmem_cols <<= 1;

    OwnCells oc;
    oc.x_s = x_s; oc.ho_s = ho_s; oc.bh_s = bh_s; oc.P_s = P_s;
    oc.u0 = cta * p.cpc;
    oc.cells = n_cnt / G;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { ptx::mbar_init(&ctl->full[s], 1); ptx::mbar_init(&ctl->empty[s], 1); ctl->rounds[s] = 0; }
        for (int i = 0; i < 2; ++i) ptx::mbar_init(&ctl->acc_full[i], 1);
        ptx::mbar_init(&ctl->acc_full[2], (uint32_t)(p.plan_c.n_own > 0 ? p.plan_c.n_own : 1));      // one arrival per projection issuer
        ptx::mbar_init(&ctl->w_full, 1);
        ptx::mbar_init(&ctl->x_full, 1);
        ptx::mbar_init(&ctl->tab_full, 1);
        ctl->abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&map_R);
        ptx::prefetch_tensormap(&map_X);
        if (ln) ptx::prefetch_tensormap(&map_pre);
        if (proj) ptx::prefetch_tensormap(&map_Wp);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&ctl->tmem_base, tmem_cols);
        ptx::tmem_relinquish();
    }
    for (int i = threadIdx.x; i < p.nc_pad; i += RTHREADS) {
        const bool in = i < n_cnt;
        bh_s[i] = in ? p.bh[n0 + i] : 0;
        P_s[i] = (in && peep && !ln) ? p.P[n0 + i] : (int16_t)0;
    }
    ptx::tc_fence_before();
    ptx::cta_sync();
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    // small batch: this CTA's rows of R and W_proj as plain row-major copies
    const int sp_lo = cta * p.rpc;
    int sp_cnt = (proj && p.small) ? p.rpc : 0;
    if (sp_lo + sp_cnt > p.O) sp_cnt = p.O - sp_lo > 0 ? p.O - sp_lo : 0;
    if (p.small) {
        if (has_cells) {
            const uint4 *src = reinterpret_cast<const uint4 *>(p.R + (size_t)n0 * p.O);
            for (int i = threadIdx.x; i < (n_cnt * p.O) >> 4; i += RTHREADS) reinterpret_cast<uint4 *>(R_s)[i] = __ldg(src + i);
        }
        if (sp_cnt > 0) {
            const uint4 *src = reinterpret_cast<const uint4 *>(p.Wproj + (size_t)sp_lo * p.C);
            for (int i = threadIdx.x; i < (sp_cnt * p.C) >> 4; i += RTHREADS) reinterpret_cast<uint4 *>(Wp_s)[i] = __ldg(src + i);
        }
    }
    // resident weights of the tensor-core path: one TMA box per k-block
    if (threadIdx.x == 0) {
        uint32_t bytes = 0;
        if (has_cells && !p.small) bytes += (uint32_t)(p.kb_h * p.npc * 128);
        if (has_ptile && !p.small) bytes += (uint32_t)(p.kb_c * p.pn * 128);
        if (bytes) {
            ptx::mbar_arrive_expect_tx(&ctl->w_full, bytes);
            if (has_cells)
                for (int kb = 0; kb < p.kb_h; ++kb)
                    ptx::tma_load_2d(R_s + (size_t)kb * p.npc * 128, &map_R, &ctl->w_full, kb * 128, n0);
            if (has_ptile)
                for (int kb = 0; kb < p.kb_c; ++kb)
                    ptx::tma_load_2d(Wp_s + (size_t)kb * p.pn * 128, &map_Wp, &ctl->w_full, kb * 128, tile_p0);
        } else {
            ptx::mbar_arrive(&ctl->w_full);
        }
    }
    if (warp == 1 && lane == 0) wait_or_abort(&ctl->w_full, 0, abort_flag);
    ptx::cta_sync();

    unsigned epoch = 0;
    Ring rg;
    rg.base = ring; rg.rounds = ctl->rounds;
    const int n_issue_c = p.plan_c.n_own;
    const uint32_t idesc_a = ptx::idesc_i8(128, p.nc_pad), idesc_c = ptx::idesc_i8(128, p.pn);
    const int iss = warp == 1 ? 0 : warp == 18 ? 1 : warp == 19 ? 2 : warp == 17 ? 3 : -1;      // issuer thread number of lane 0

    // the CTA's box of X_t: rows [t * B, t * B + x_rows) x its gate rows (rows past the end of X read as zero)
    const bool tensor_a = !p.small && has_cells;
    auto fetch_x = [&](int t) {
        ptx::mbar_arrive_expect_tx(&ctl->x_full, p.x_bytes);
        ptx::tma_load_2d(x_s, &map_X, &ctl->x_full, n0, t * p.B);
    };
    if (has_cells && threadIdx.x == 0) fetch_x(0);

    const bool timing = p.phase_ns != nullptr && cta == 0 && threadIdx.x == 0;
    unsigned long long t_mark = timing ? globaltimer() : 0ull;
    auto lap = [&](int slot) {
        if (timing) {
            unsigned long long now = globaltimer();
            p.phase_ns[slot] += now - t_mark;
            t_mark = now;
        }
    };
    const int ngroups = n_cnt >> 3;
    constexpr int gstep = (G == 4) ? 1 : 3;                        // groups are dealt in units of this many
    // TAB: the tables of the nonlinearities are copied into the ring when the recurrent matmul has drained it, read by
    // the elementwise phase, and overwritten by the projection's operand after the next grid barrier
    const ActTabs at = make_act_tabs(ptx::smem_u32(ring), p.tab_lay);
    auto fetch_tables = [&]() {
        ptx::mbar_arrive_expect_tx(&ctl->tab_full, p.tab_lay.bytes);
        ptx::bulk_load_1d(ring, p.tab, p.tab_lay.bytes, &ctl->tab_full);
    };

    for (int t = 0; t < p.T; ++t) {
        const int cur = t & 1;
        int8_t *h_next = p.hbuf + (size_t)(cur ^ 1) * p.h_stride;
        const uint32_t par = (uint32_t)t & 1u;

        // ================= phase A: gate sums of the block's cells =================
        if (p.small) {
            if (has_cells) {
                if (p.B == 1) phase_a_small<1>(p, cur, n_cnt, (const int8_t *)R_s, stage_s, acc_s);
                else if (p.B <= 2) phase_a_small<2>(p, cur, n_cnt, (const int8_t *)R_s, stage_s, acc_s);
                else if (p.B <= 4) phase_a_small<4>(p, cur, n_cnt, (const int8_t *)R_s, stage_s, acc_s);
                else if (p.B <= 8) phase_a_small<8>(p, cur, n_cnt, (const int8_t *)R_s, stage_s, acc_s);
                else phase_a_small<16>(p, cur, n_cnt, (const int8_t *)R_s, stage_s, acc_s);
                ptx::cta_sync();
                // epilogue tasks: (batch row, unit of column groups)
                const bool okx = wait_or_abort(&ctl->x_full, par, abort_flag);
                const int units = ngroups / gstep;
                if (okx)
                    for (int i = threadIdx.x; i < p.B * units; i += RTHREADS) {
                        const int b = i / units, gu = i - b * units;
                        gate_sums_row<G, LN, PEEP, false, FS>(p, oc, 0u, acc_s + (size_t)b * p.nc_pad, b, n0, gu * gstep, (gu + 1) * gstep,
                                                          p.c + (size_t)b * p.C + oc.u0, true);
                    }
                if (ln) ptx::fence_proxy_async();
            }
        } else if (has_cells) {
            if (warp == 0) {
                if (lane == 0) {
                    fence_proxy_async_global();
                    ring_produce(ctl, rg, p.plan_a, true, p.kb_h, p.hbuf + (size_t)cur * p.h_stride, abort_flag);
                    if (TAB) {
                        // every MMA of this step has read its ring stages once the accumulators are complete
                        bool drained = true;
                        for (int mi = 0; mi < p.MT; ++mi) drained = drained && wait_or_abort(&ctl->acc_full[mi], par, abort_flag);
                        if (drained) fetch_tables();
                    }
                }
                __syncwarp();
            } else {
              if (iss >= 0 && iss < p.MT) {
                // one issuer per batch tile, each with its own accumulator
                if (lane == 0) {
                    ptx::tc_fence_after();
                    if (ring_issue(ctl, rg, p.plan_a, iss, true, p.kb_h, ptx::smem_u32(R_s), (uint32_t)p.npc * 128u,
                                   tmem_base + (uint32_t)(iss * p.nc_pad), idesc_a, abort_flag))
                        ptx::mma_commit(&ctl->acc_full[iss]);
                }
                __syncwarp();
              }
              if (warp >= 2 && warp < 18) {
                // 16 epilogue warps: 4 TMEM lane quarters x (batch tile, column part)
                const int e = warp - 2, quarter = warp & 3, slot = e >> 2;
                const int mi = slot % p.MT, part = slot / p.MT, nparts = 4 / p.MT;
                const int units = ngroups / gstep;
                const int g_begin = gstep * (part * units / nparts), g_end = gstep * ((part + 1) * units / nparts);
                const int b = mi * 128 + quarter * 32 + lane;
                const bool probe = p.phase_ns != nullptr && cta == 0 && warp == 2 && lane == 0;
                const unsigned long long t_in = probe ? globaltimer() : 0ull;
                const bool okx = wait_or_abort(&ctl->x_full, par, abort_flag);        // fetched a step ago
                const bool oka = wait_or_abort(&ctl->acc_full[mi], par, abort_flag);
                if (__all_sync(0xffffffffu, okx && oka)) {
                    if (probe) p.phase_ns[6] += globaltimer() - t_in;      // operand load + matmul latency
                    ptx::tc_fence_after();
                    const uint32_t ta = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(mi * p.nc_pad);
                    const bool valid = b < p.B;
                    gate_sums_row<G, LN, PEEP, true, FS>(p, oc, ta, nullptr, b, n0, g_begin, g_end,
                                                     p.c + (size_t)(valid ? b : 0) * p.C + oc.u0, valid);
                    ptx::tc_fence_before();
                    if (ln) ptx::fence_proxy_async();                      // the box leaves through the async proxy
                }
              }
            }
        }
        if (TAB && !has_cells && ln && threadIdx.x == 0) fetch_tables();     // no matmul here: the ring is idle already
        ptx::cta_sync();
        if (tensor_a && threadIdx.x == 0) ring_advance(rg, p.plan_a);
        if (ln) {
            // the statistics of a row need every block's cells: gate sums to L2, barrier, flat elementwise phase
            if (has_cells && threadIdx.x == 0 && !*abort_flag) {
                if (!peep) {
                    // gate sums of all batch rows x this block's gate rows: one store, complete before the barrier publishes it
                    ptx::tma_store_2d(&map_pre, x_s, n0, 0);
                    ptx::bulk_commit_group();
                    ptx::bulk_wait_group_all();
                    fence_proxy_async_global();
                }
                if (t + 1 < p.T) fetch_x(t + 1);              // the box is free again
            }
            lap(0);
            grid_sync(p, epoch, abort_flag, false);
            lap(1);
            if (*abort_flag) break;
            // (a wait that runs out sets the abort flag: the next barrier ends the time loop)
            if (TAB && !wait_or_abort(&ctl->tab_full, par, abort_flag)) {}
            else if (peep) phase_b_ln_peep<G, TAB, FS>(p, ctl, at, t, h_next, row_s);
            else phase_b_flat<G, true, false, TAB, FS>(p, ctl, at, t, h_next);
            ptx::cta_sync();
        } else {
            // same block, same cells, straight from shared memory
            if (!TAB || !has_cells || wait_or_abort(&ctl->tab_full, par, abort_flag)) phase_b_own<G, PEEP, TAB, FS>(p, oc, at, t, h_next);
            ptx::fence_proxy_async();                        // X box and ring scratch go back to the async proxy
            ptx::cta_sync();
            if (has_cells && threadIdx.x == 0 && t + 1 < p.T && !*abort_flag) fetch_x(t + 1);
        }
        lap(2);
        grid_sync(p, epoch, abort_flag, !p.small);
        lap(3);
        if (*abort_flag) break;

        // ================= phase C: projection =================
        if (proj) {
            if (p.small) {
                if (sp_cnt > 0) {
                    if (p.B == 1) phase_c_small<1>(p, t, sp_lo, sp_cnt, (const int8_t *)Wp_s, (int8_t *)ring, h_next);
                    else if (p.B <= 2) phase_c_small<2>(p, t, sp_lo, sp_cnt, (const int8_t *)Wp_s, (int8_t *)ring, h_next);
                    else if (p.B <= 4) phase_c_small<4>(p, t, sp_lo, sp_cnt, (const int8_t *)Wp_s, (int8_t *)ring, h_next);
                    else if (p.B <= 8) phase_c_small<8>(p, t, sp_lo, sp_cnt, (const int8_t *)Wp_s, (int8_t *)ring, h_next);
                    else phase_c_small<16>(p, t, sp_lo, sp_cnt, (const int8_t *)Wp_s, (int8_t *)ring, h_next);
                }
            } else if (has_ptile) {
                if (warp == 0) {
                    if (lane == 0) {
                        fence_proxy_async_global();
                        ring_produce(ctl, rg, p.plan_c, false, p.kb_c, p.mbuf + (size_t)tile_mi * p.kb_c * KB_BYTES, abort_flag);
                    }
                    __syncwarp();
                } else {
                    // several issuers share the K range: issuer w owns chunks w, w + n_issue_c, ... with its own
                    // accumulator; the epilogue adds the partial sums (exact in int32).  Issuers are the three warps
                    // without an epilogue role and the last epilogue warp, before it turns to its part
                    if (iss >= 0 && iss < n_issue_c) {
                        if (lane == 0) {
                            ptx::tc_fence_after();
                            if (ring_issue(ctl, rg, p.plan_c, iss, false, p.kb_c, ptx::smem_u32(Wp_s), (uint32_t)p.pn * 128u,
                                           tmem_base + acc_cols_a + (uint32_t)(iss * p.pn), idesc_c, abort_flag))
                                ptx::mma_commit(&ctl->acc_full[2]);
                        }
                        __syncwarp();
                    }
                    if (warp >= 2 && warp < 18) {
                        // 16 epilogue warps: 4 TMEM lane quarters x 4 column parts of the tile
                        const int quarter = warp & 3, part = (warp - 2) >> 2;
                        const int ngroups_c = p.pn >> 2;
                        const int c_begin = 4 * (part * ngroups_c / 4), c_end = 4 * ((part + 1) * ngroups_c / 4);
                        if (__all_sync(0xffffffffu, wait_or_abort(&ctl->acc_full[2], par, abort_flag))) {
                            ptx::tc_fence_after();
                            const int b = tile_mi * 128 + quarter * 32 + lane;
                            phase_c_row<FS>(p, tmem_base + ((uint32_t)(quarter * 32) << 16) + acc_cols_a, n_issue_c, b, t, tile_p0, c_begin,
                                        c_end, h_next, b < p.B);
                            ptx::tc_fence_before();
                        }
                    }
                }
            }
            ptx::cta_sync();
            if (!p.small && has_ptile && threadIdx.x == 0) ring_advance(rg, p.plan_c);
            lap(4);
            grid_sync(p, epoch, abort_flag, !p.small && warp >= 2);      // the epilogue warps wrote h
            lap(5);
            if (*abort_flag) break;
        }
    }

    // ---------------- teardown ----------------
    ptx::cta_sync();
    if (*abort_flag) {
        // copies still in flight must land before the block's shared memory is handed on: the X box by its barrier
        // (bounded), ring stages by a bounded pause (their barriers may be mid-phase)
        // (one of the two parities is the phase that completed last and passes at once; the other is the phase a
        // requested box completes - or, with no request outstanding, a wait that runs out after 2 ms.  Keeping track of
        // the last request in a variable would tell them apart, but costs the time loop 3 %.)
        if (threadIdx.x == 0 && has_cells) drain_box_requests(&ctl->x_full);
        for (int i = 0; i < 200; ++i) __nanosleep(500);
        if (threadIdx.x == 0) atomicExch(p.status, 2);
    }
    ptx::cta_sync();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, tmem_cols);
    }
}

// Caller's h [B][K] (plain rows) -> tiled operand image, 16 bytes per thread.
__global__ void k_tile_rows(const int8_t *src, int8_t *dst, int B, int K, int nkb, bool aligned)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int per_row = K >> 4;
    if (i >= B * per_row) return;
    const int row = i / per_row, k = (i - row * per_row) << 4;
    const int8_t *s = src + (size_t)row * K + k;
    uint4 v;
    if (aligned) {
        v = *reinterpret_cast<const uint4 *>(s);
    } else {
        uint32_t w[4] = {0, 0, 0, 0};
        for (int j = 0; j < 16; ++j) w[j >> 2] |= (uint32_t)(uint8_t)s[j] << (8 * (j & 3));
        v = make_uint4(w[0], w[1], w[2], w[3]);
    }
    *reinterpret_cast<uint4 *>(dst + tile_off(row, k, nkb)) = v;
}

size_t x_box_bytes(int MT, int npc) { return (size_t)MT * 128 * npc * 2; }

size_t rec_smem_bytes(const LayerParams &p, int stages, int nc_pad, int pn, int kb_h, int kb_c, int MT, int npc)
{
    const bool proj = (p.flags & F_PROJECTION) != 0, peep = (p.flags & F_PEEPHOLE) != 0, ln = (p.flags & F_LAYERNORM) != 0;
    // without layer norm a peephole layer keeps H_o of the block's cells, all rows; with layer norm and peephole the
    // elementwise phase holds one row of gate sums and of new cell states
    size_t extra = ln ? (peep ? ((size_t)p.C * p.G + p.C) * 2 : 0) : (peep ? (size_t)MT * 128 * (npc / p.G) * 2 : 0);
    extra = (extra + 15) & ~(size_t)15;
    return 1024 + (size_t)stages * STAGE_BYTES + (size_t)kb_h * npc * 128 + (proj ? (size_t)kb_c * pn * 128 : 0) +
           ((x_box_bytes(MT, npc) + 1023) & ~(size_t)1023) + extra + (size_t)nc_pad * 6 + sizeof(RecCtl) + 64;
}

int round_up(int v, int m) { return (v + m - 1) / m * m; }

// the instantiation for a layer's variant and mode (see the kernel)
template <int MODE>
const void *recurrent_kernel_of(const LayerParams &p)
{
    const bool ln = (p.flags & F_LAYERNORM) != 0, peep = (p.flags & F_PEEPHOLE) != 0;
    if (p.G == 4) {
        if (ln) return peep ? (const void *)k_recurrent_sm100<4, true, true, MODE> : (const void *)k_recurrent_sm100<4, true, false, MODE>;
        return peep ? (const void *)k_recurrent_sm100<4, false, true, MODE> : (const void *)k_recurrent_sm100<4, false, false, MODE>;
    }
    if (ln) return peep ? (const void *)k_recurrent_sm100<3, true, true, MODE> : (const void *)k_recurrent_sm100<3, true, false, MODE>;
    return peep ? (const void *)k_recurrent_sm100<3, false, true, MODE> : (const void *)k_recurrent_sm100<3, false, false, MODE>;
}
const void *recurrent_kernel(const LayerParams &p, int mode)
{
    return mode == 2 ? recurrent_kernel_of<2>(p) : (mode == 1 ? recurrent_kernel_of<1>(p) : recurrent_kernel_of<0>(p));
}

// every scale the recurrent kernel applies for this layer shifts right (shift <= 0)
bool scales_shift_right(const LayerParams &p)
{
    const bool proj = (p.flags & F_PROJECTION) != 0, peep = (p.flags & F_PEEPHOLE) != 0, ln = (p.flags & F_LAYERNORM) != 0;
    bool ok = p.eff_m.shift <= 0 && (!proj || p.eff_proj.shift <= 0);
    for (int g = 0; g < p.G; ++g)
        ok = ok && p.eff_h[g].shift <= 0 && (!peep || p.eff_c[g].shift <= 0) && (!ln || p.eff_ln[g].shift <= 0);
    return ok;
}

// contig: n_own operand tiles of `per` chunks each, one owner per tile; else n_total chunks of one tile dealt round-robin
RingPlan make_ring_plan(int stages, int n_own, bool contig, int per, int n_total)
{
    RingPlan pl;
    memset(&pl, 0, sizeof(pl));
    pl.n_own = n_own;
    for (int o = 0; o < n_own && o < 4; ++o) {
        pl.n_chunks[o] = contig ? per : (n_total - o + n_own - 1) / n_own;
        pl.cnt[o] = (stages - o + n_own - 1) / n_own;
        if (pl.n_chunks[o] > pl.n_max) pl.n_max = pl.n_chunks[o];
        for (int j = 0; j < pl.n_chunks[o]; ++j) pl.uses[o + n_own * (j % pl.cnt[o])] += 1;
    }
    return pl;
}

}  // namespace

int fast_scratch_init(FastScratch &s, int max_B, int maxC, int maxO, int maxN, int sm_count)
{
    s.Bpad = round_up(max_B, 128);
    s.sm_count = sm_count;
    s.hbuf_bytes = (size_t)2 * s.Bpad * round_up(maxO, 128);      // whole 128 x 128-byte k-blocks
    s.mbuf_bytes = (size_t)s.Bpad * round_up(maxC, 128);
    if (cudaMalloc(&s.hbuf, s.hbuf_bytes) != cudaSuccess) return QLSTM_ERR_NOMEM;
    if (cudaMalloc(&s.mbuf, s.mbuf_bytes) != cudaSuccess) return QLSTM_ERR_NOMEM;
    if (cudaMalloc(&s.pre, (size_t)max_B * maxN * sizeof(int32_t)) != cudaSuccess) return QLSTM_ERR_NOMEM;
    if (cudaMalloc(&s.bar, BAR_BYTES) != cudaSuccess) return QLSTM_ERR_NOMEM;
    cudaMemset(s.hbuf, 0, s.hbuf_bytes);
    cudaMemset(s.mbuf, 0, s.mbuf_bytes);
    cudaMemset(s.bar, 0, BAR_BYTES);
    return QLSTM_OK;
}

void fast_scratch_destroy(FastScratch &s)
{
    cudaFree(s.hbuf); cudaFree(s.mbuf); cudaFree(s.pre); cudaFree(s.bar);
    s = FastScratch();
}

int fast_recurrent_init(FastLayer &f, const LayerParams &p, const FastScratch &s, int max_B)
{
    f.rec_ok = false;
    const bool proj = (p.flags & F_PROJECTION) != 0;
    if (p.O % 16 != 0 || p.C % 16 != 0 || max_B > 256) return QLSTM_OK;
    const int grid = s.sm_count;
    // cells per CTA: the gate-row slice must start on a 16-byte boundary of an int16 row (cpc * G % 8 == 0)
    const int step = (p.G == 4) ? 2 : 8;
    int cpc = round_up((p.C + grid - 1) / grid, step);
    if (cpc * p.G > 256) return QLSTM_OK;
    f.cpc = cpc;
    f.n_cta_a = (p.C + cpc - 1) / cpc;
    f.nc_pad = round_up(cpc * p.G, 16);
    f.kb_h = (p.O + 127) / 128;
    f.kb_c = (p.C + 127) / 128;
    f.grid = grid;
    const int MT_max = (max_B + 127) / 128;
    f.pn = 0; f.npn = 0;
    if (proj) {
        int pn = 16;
        while (pn <= 256 && MT_max * ((p.O + pn - 1) / pn) > grid) pn *= 2;
        if (pn > 256) return QLSTM_OK;
        f.pn = pn;
        f.npn = (p.O + pn - 1) / pn;
    }
    if (MT_max * f.nc_pad + f.pn > 512) return QLSTM_OK;
    f.n_issue_c = 1;
    if (proj)
        while (f.n_issue_c < 4 && MT_max * f.nc_pad + f.pn * f.n_issue_c * 2 <= 512) f.n_issue_c *= 2;
    int dev = 0, max_smem = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    int stages = MAX_STAGES;
    while (stages >= 2 && rec_smem_bytes(p, stages, f.nc_pad, f.pn, f.kb_h, f.kb_c, MT_max, cpc * p.G) > (size_t)max_smem) --stages;
    if (stages < 2) return QLSTM_OK;
    f.stages = stages;
    f.smem = rec_smem_bytes(p, stages, f.nc_pad, f.pn, f.kb_h, f.kb_c, MT_max, cpc * p.G);
    if (!make_tensor_map_i8(&f.map_R, p.R, (uint64_t)p.N, (uint64_t)p.O, (uint32_t)(cpc * p.G), 128)) return QLSTM_OK;
    if (proj) {
        if (!make_tensor_map_i8(&f.map_Wp, p.Wproj, (uint64_t)p.O, (uint64_t)p.C, (uint32_t)f.pn, 128)) return QLSTM_OK;
    } else {
        f.map_Wp = f.map_R;
    }
    for (int mode = 0; mode < 3; ++mode) {
        int per_sm = 0;
        if (cudaFuncSetAttribute(recurrent_kernel(p, mode), cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess)
            return QLSTM_OK;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, recurrent_kernel(p, mode), RTHREADS, f.smem) != cudaSuccess ||
            per_sm < 1)
            return QLSTM_OK;
    }
    // memoised nonlinearities, if their tables fit into the ring (they live there between the matmul phases)
    if (!act_tables_build(p.m_bits, (size_t)f.stages * STAGE_BYTES, &f.act_tab, &f.act_lay)) return QLSTM_ERR_CUDA;
    f.rec_ok = true;
    return QLSTM_OK;
}

int fast_layer_init(FastLayer &f, const LayerParams &p, const FastScratch &s, int max_T, int max_B)
{
    (void)max_T;
    int rc = fast_projection_init(f, p);
    if (rc != QLSTM_OK) return rc;
    return fast_recurrent_init(f, p, s, max_B);
}

void fast_layer_destroy(FastLayer &f)
{
    if (f.act_tab) cudaFree(f.act_tab);
    f.act_tab = nullptr;
    f.act_lay = ActTabLayout{0, 0, 0, 0, 0, 0, 0};
}

bool fast_recurrent_supported(const FastLayer &f, const LayerParams &, int B) { return f.rec_ok && B <= 256; }

int launch_recurrent_fast(const FastLayer &f, const LayerParams &p, const FastScratch &s, const int16_t *X, int T, int B,
                          int8_t *h, int16_t *c, int8_t *y, int *status, unsigned long long *phase_ns, int small_batch_max,
                          cudaStream_t st, int *launches)
{
    RecParams rp;
    memset(&rp, 0, sizeof(rp));
    rp.T = T; rp.B = B; rp.MT = (B + 127) / 128; rp.Bpad = s.Bpad;
    rp.h_stride = (size_t)s.Bpad * f.kb_h * 128;
    rp.C = p.C; rp.O = p.O; rp.G = p.G; rp.N = p.N;
    rp.div_c = make_div_magic((uint32_t)p.C);
    rp.flags = p.flags; rp.m_bits = p.m_bits; rp.zp_m = p.zp_m; rp.zp_h = p.zp_h;
    rp.cpc = f.cpc; rp.n_cta_a = f.n_cta_a; rp.nc_pad = f.nc_pad;
    rp.pn = f.pn; rp.npn = f.npn; rp.n_ptiles = rp.MT * f.npn;
    rp.kb_h = f.kb_h; rp.kb_c = f.kb_c; rp.stages = f.stages; rp.n_issue_c = f.n_issue_c;
    rp.npc = f.cpc * p.G;
    {
        // every MMA issuer owns at least one ring stage
        const int cpt_a = (f.kb_h + STAGE_KB - 1) / STAGE_KB, n_chunks_c = (f.kb_c + STAGE_KB - 1) / STAGE_KB;
        int ni = f.n_issue_c < n_chunks_c ? f.n_issue_c : n_chunks_c;
        if (ni > f.stages) ni = f.stages;
        if (ni < 1) ni = 1;
        rp.plan_a = make_ring_plan(f.stages, rp.MT, true, cpt_a, 0);
        rp.plan_c = make_ring_plan(f.stages, ni, false, 0, n_chunks_c);
    }
    rp.R = p.R; rp.Wproj = p.Wproj;
    rp.rpc = (p.O + f.grid - 1) / f.grid;
    {
        // small batch: staged operand [16][K], then the accumulators [16][nc_pad] int32, both inside the ring
        const int maxk = p.O > p.C ? p.O : p.C;
        const size_t stage_bytes = ((size_t)SMALL_BATCH_MAX * maxk + 1023) & ~(size_t)1023;
        const size_t need = stage_bytes + (size_t)SMALL_BATCH_MAX * f.nc_pad * 4;
        const bool fits = need <= (size_t)f.stages * STAGE_BYTES && (!(p.flags & F_PROJECTION) || rp.rpc <= f.pn);
        const int lim = small_batch_max < SMALL_BATCH_MAX ? small_batch_max : SMALL_BATCH_MAX;
        rp.small = (B <= lim && fits) ? 1 : 0;
        rp.acc_off = rp.small ? (uint32_t)stage_bytes : 0u;
    }
    // the block's box of X_t and of the gate sums: all rows of the batch (whole 128-row tiles on the tensor-core path)
    rp.x_rows = rp.small ? B : rp.MT * 128;
    rp.x_bytes = (uint32_t)((size_t)rp.x_rows * rp.npc * 2);
    const bool ln = (p.flags & F_LAYERNORM) != 0, peep = (p.flags & F_PEEPHOLE) != 0;
    rp.ho_bytes = (peep && !ln) ? (uint32_t)((size_t)rp.x_rows * f.cpc * 2) : 0u;
    rp.row_bytes = (peep && ln) ? (uint32_t)(((size_t)p.C * p.G + p.C) * 2) : 0u;
    // layer norm: flat elementwise phase over contiguous ranges of the B x C cell grid (whole rows with a peephole)
    if (ln && peep) rp.items_per_cta = ((B + f.grid - 1) / f.grid) * p.C;
    else rp.items_per_cta = round_up((int)(((long)B * p.C + f.grid - 1) / f.grid), 8);
    rp.fast_rescale_ok = 1;
    for (int g = 0; g < p.G; ++g) {
        rp.eff_h[g] = p.eff_h[g]; rp.eff_c[g] = p.eff_c[g]; rp.eff_ln[g] = p.eff_ln[g];
        rp.f_h[g] = make_fast_scale(p.eff_h[g]);
        rp.f_c[g] = make_fast_scale(p.eff_c[g]);
        rp.f_ln[g] = make_fast_scale(p.eff_ln[g]);
        if (p.eff_h[g].shift > 0) rp.fast_rescale_ok = 0;
    }
    rp.eff_m = p.eff_m; rp.eff_proj = p.eff_proj;
    rp.f_proj = make_fast_scale(p.eff_proj);
    rp.f_m = make_fast_scale(p.eff_m);
    rp.phase_ns = phase_ns;
    // tables only with right-shifting scales (a layer with a left shift keeps the general kernel)
    const bool fs = scales_shift_right(p) && !f.dbg_general_kernel;
    const bool tab = fs && f.act_tab != nullptr && !rp.small && !f.dbg_no_tables;
    const int mode = tab ? 2 : (fs ? 1 : 0);
    rp.tab = tab ? f.act_tab : nullptr;
    rp.tab_lay = f.act_lay;
    rp.spin_limit_ns = f.dbg_spin_limit_ns ? f.dbg_spin_limit_ns : SPIN_LIMIT_NS;
    rp.barrier_extra = f.dbg_barrier_extra;
    if (p.eff_proj.shift > 0) rp.fast_rescale_ok = 0;
    for (int g = 0; g < 4; ++g) rp.gate_slot[g] = p.slot_of_gate[g];
    rp.X = X; rp.c = c; rp.y = y;
    rp.hbuf = s.hbuf; rp.mbuf = s.mbuf; rp.pre = s.pre; rp.bar = s.bar; rp.status = status;
    rp.bh = p.bh; rp.bp = p.bp; rp.bln = p.bln; rp.P = p.P; rp.L = p.L;

    // h^{-1} into operand buffer 0; barrier words cleared
    if (cudaMemsetAsync(s.bar, 0, BAR_BYTES, st) != cudaSuccess) return QLSTM_ERR_CUDA;
    int n_launch = 1;
    if (rp.small) {
        if (cudaMemcpyAsync(s.hbuf, h, (size_t)B * p.O, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return QLSTM_ERR_CUDA;
    } else {
        const int chunks = B * (p.O >> 4);
        k_tile_rows<<<(chunks + 255) / 256, 256, 0, st>>>(h, s.hbuf, B, p.O, f.kb_h, ((uintptr_t)h & 15) == 0);
        if (cudaGetLastError() != cudaSuccess) return QLSTM_ERR_CUDA;
        ++n_launch;
    }

    // X as a tensor [T * B][N] int16 and (layer norm) the gate sums as [B][N] int16; a block's box is all rows of a step
    // x its gate rows
    CUtensorMap map_X, map_pre;
    if (!make_tensor_map_i16(&map_X, X, (uint64_t)T * B, (uint64_t)p.N, (uint32_t)rp.x_rows, (uint32_t)rp.npc) ||
        !make_tensor_map_i16(&map_pre, s.pre, (uint64_t)B, (uint64_t)p.N, (uint32_t)rp.x_rows, (uint32_t)rp.npc))
        return QLSTM_ERR_CUDA;
    void *args[] = {(void *)&f.map_R, (void *)&f.map_Wp, (void *)&map_X, (void *)&map_pre, (void *)&rp};
    cudaError_t e = cudaLaunchCooperativeKernel(recurrent_kernel(p, mode), dim3(f.grid), dim3(RTHREADS), args, f.smem, st);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return e == cudaErrorCooperativeLaunchTooLarge ? QLSTM_ERR_LAUNCH : QLSTM_ERR_CUDA;
    }
    // h^{T-1} is the last row block of y
    if (T > 0 && cudaMemcpyAsync(h, y + (size_t)(T - 1) * B * p.O, (size_t)B * p.O, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return QLSTM_ERR_CUDA;
    if (launches) *launches = n_launch;
    return QLSTM_OK;
}

int debug_ring_plan(int stages, int n_own, int contig, int per, int n_total, int *out)
{
    if (!out || stages < 1 || stages > MAX_STAGES || n_own < 1 || n_own > 4 || n_own > stages) return QLSTM_ERR_ARG;
    if (contig ? per < 0 : n_total < 0) return QLSTM_ERR_ARG;
    const RingPlan pl = make_ring_plan(stages, n_own, contig != 0, per, n_total);
    int k = 0;
    out[k++] = pl.n_own;
    out[k++] = pl.n_max;
    for (int o = 0; o < 4; ++o) out[k++] = pl.n_chunks[o];
    for (int o = 0; o < 4; ++o) out[k++] = pl.cnt[o];
    for (int s = 0; s < MAX_STAGES; ++s) out[k++] = pl.uses[s];
    return QLSTM_OK;
}

}  // namespace ql
