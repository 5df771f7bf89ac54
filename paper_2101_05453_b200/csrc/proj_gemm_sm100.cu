// Batched input projection on the 5th-generation tensor cores (Section 3.2.4, first rescale term):
//
//   X[r][n] = sat16( rescale( sum_j W[n][j] * x[r][j] + bx[n], eff_x[gate(n)] ) ),   r < rows, n < N = C*G
//
// int8 x int8 -> int32 dense contraction, so it runs as tcgen05.mma kind::i8 with the int32
// accumulator in tensor memory.  The rescale to int16 is fused into the epilogue: writing int32
// accumulators would double the HBM traffic of a kernel whose output already costs as much time
// as its math (K is only 512-1024).
//
// With K this small a 128 x 256 output tile needs 240 KB of operands for 42 MOP: streaming both
// operands per tile is bound by L2 -> SM bandwidth, not by the tensor cores.  So the weight panel
// (BN rows of W, all of K) stays resident in shared memory while the CTA walks down the M tiles of
// that panel; only the x tile (128 x K bytes) is streamed per output tile.
//
// One persistent CTA per SM, warp specialised:
//   warp 0       TMA producer: W panel [BN x K] once per panel; x k-blocks [128 x 128 B] through a ring
//   warp 1       MMA issuer:   4 x (M128 N=BN K32) per k-block into one of two TMEM accumulators
//   warps 2..17  epilogue:     tcgen05.ld -> + folded bias -> fixed-point rescale -> sat16 -> stores,
//                              overlapping the next tile's MMAs through the second TMEM accumulator
// Tiles are numbered panel-major.  Where the SMs hold at least one CTA per panel, CTA b keeps panel
// b % panels for the whole launch and walks one of floor(SMs / panels) ranges of M tiles; the CTAs of a
// range then ask for the same x tiles at about the same time, so x reaches L2 from HBM once instead of
// once per panel (the int16 output, 2 N / K times the size of x, would otherwise push it out between
// uses).  The panel width is chosen so that panels x ranges fills the SMs.  Otherwise the tiles are
// split into equal contiguous ranges and a CTA touches at most two panels.  x is loaded with an L2
// evict-last hint and the output stored with evict-first.  No cluster launch and no multicast.
#include "../../include/qlstm.h"
#include "../../include/qlstm_debug.h"
#include "fast_kernels.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace ql {

namespace {

constexpr int BM = 128, BK = 128, MAX_STAGES = 6, EPI_WARPS = 16;
constexpr int A_BYTES = BM * BK;
constexpr int THREADS = 32 * (2 + EPI_WARPS);
constexpr int TMEM_COLS = 512;
constexpr int W_BYTES_MAX = 160 * 1024;           // resident weight panel
constexpr int BIAS_PER_WARP = 64;                 // two 32-column chunks per epilogue warp

struct ProjParams {
    int M, N, K, G;
    int bn, kb, stages;          // panel width (multiple of 32), 128-byte k-blocks, ring depth
    const int32_t *bx;
    int16_t *out;
    FastScale fs[4];
    Scale sc[4];
    int generic;                 // some gate has a positive shift: use the generic rescale
    int m_ranges;                // > 0: CTA b owns panel b % tiles_n and the m-tile range b / tiles_n of m_ranges
    int *status;
};

struct SharedCtl {
    uint64_t a_full[MAX_STAGES], a_empty[MAX_STAGES], w_full, w_free, tmem_full[2], tmem_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

// L2 eviction policies for per-access cache hints: lines touched with evict-last stay in L2 in preference to lines
// touched with evict-first.
__device__ __forceinline__ uint64_t l2_policy_evict_last()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// 2-D tiled load global -> shared with an L2 eviction policy for the lines it reads; otherwise as ptx::tma_load_2d
// (c0 is the innermost coordinate and c0 * element size a multiple of 16 bytes).
__device__ __forceinline__ void tma_load_2d_hint(void *dst, const CUtensorMap *map, uint64_t *bar, int32_t c0, int32_t c1,
                                                 uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(ptx::smem_u32(dst)), "l"((uint64_t)map), "r"(ptx::smem_u32(bar)), "r"(c0), "r"(c1), "l"(policy)
        : "memory");
}

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

// 16 adjacent columns of one output row: + folded bias -> rescale -> sat16 -> one 32-byte store.
// fs / sc hold the gates' scales in the order of the columns of the warp's first piece: slot k is the gate of
// its column k.  Pieces are 16 columns wide, so piece `piece` starts piece slots later (16 = 1 mod 3, 0 mod 4) and
// column j of it takes slot (piece + j) % 3, or j % 4: a constant once the piece loop is unrolled.
template <int G, bool GENERIC>
__device__ __forceinline__ void epilogue_piece(const uint32_t (&r)[16], const int32_t *bias, const FastScale (&fs)[4],
                                               const Scale (&sc)[4], int piece, int16_t *dst, int n_valid, bool wide_ok,
                                               uint64_t st_policy)
{
    uint32_t packed[8];
#pragma unroll
    for (int j = 0; j < 16; j += 4) {
        const int4 b4 = *reinterpret_cast<const int4 *>(bias + j);
        const int32_t bb[4] = {b4.x, b4.y, b4.z, b4.w};
        int32_t y[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int32_t v = (int32_t)r[j + i] + bb[i];          // |acc| + |bias| < 2^30: no overflow
            const int g = (G == 4) ? i : (piece + j + i) % 3;
            y[i] = GENERIC ? mbqm(v, sc[g]) : fast_rescale(v, fs[g]);
        }
        packed[j >> 1] = ptx::pack_sat_s16(y[0], y[1]);
        packed[(j >> 1) + 1] = ptx::pack_sat_s16(y[2], y[3]);
    }
    if (n_valid >= 16 && wide_ok) {
        // a 32-byte store fills a whole sector
        asm volatile("st.global.L2::cache_hint.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8}, %9;" ::"l"(dst), "r"(packed[0]), "r"(packed[1]),
                     "r"(packed[2]), "r"(packed[3]), "r"(packed[4]), "r"(packed[5]), "r"(packed[6]), "r"(packed[7]), "l"(st_policy)
                     : "memory");
        return;
    }
#pragma unroll
    for (int v = 0; v < 2; ++v)
        if (8 * v + 8 <= n_valid)
            *reinterpret_cast<uint4 *>(dst + 8 * v) = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
}

// G: gate slots per cell (4, or 3 with CIFG); GENERIC: some gate has a positive shift and takes the general rescale
template <int G, bool GENERIC>
__global__ void __launch_bounds__(THREADS, 1)
k_projection_sm100(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, ProjParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int w_block = p.bn * BK;                                   // bytes of one k-block of the panel
    uint8_t *W_s = smem;
    uint8_t *ring = W_s + (size_t)p.kb * w_block;
    int32_t *bias_s = (int32_t *)(ring + (size_t)p.stages * A_BYTES);
    SharedCtl *ctl = (SharedCtl *)(bias_s + EPI_WARPS * BIAS_PER_WARP);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = (p.M + BM - 1) / BM, tiles_n = (p.N + p.bn - 1) / p.bn;
    const int n_tiles = tiles_m * tiles_n;
    // Tiles are numbered panel-major.  Either every CTA takes an equal contiguous range of them, or (m_ranges > 0)
    // CTA b keeps panel b % tiles_n and walks the m-tile range b / tiles_n: the CTAs of one range then read the
    // same x tiles at about the same time, so each x tile comes from HBM once and from L2 for the other panels.
    int t_begin, t_end;
    if (p.m_ranges > 0) {
        const int n_tile = blockIdx.x % tiles_n, r = blockIdx.x / tiles_n;
        const int per = (tiles_m + p.m_ranges - 1) / p.m_ranges;
        const int mb = r * per < tiles_m ? r * per : tiles_m;
        const int me = mb + per < tiles_m ? mb + per : tiles_m;
        t_begin = n_tile * tiles_m + mb;
        t_end = n_tile * tiles_m + me;
    } else {
        const int per_cta = (n_tiles + gridDim.x - 1) / gridDim.x;
        t_begin = blockIdx.x * per_cta;
        t_end = (t_begin + per_cta < n_tiles) ? t_begin + per_cta : n_tiles;
    }
    volatile int *abort_flag = &ctl->abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { ptx::mbar_init(&ctl->a_full[s], 1); ptx::mbar_init(&ctl->a_empty[s], 1); }
        ptx::mbar_init(&ctl->w_full, 1);
        ptx::mbar_init(&ctl->w_free, 1);
        for (int b = 0; b < 2; ++b) { ptx::mbar_init(&ctl->tmem_full[b], 1); ptx::mbar_init(&ctl->tmem_empty[b], EPI_WARPS); }
        ctl->abort_flag = 0;
        ptx::fence_barrier_init();
        ptx::prefetch_tensormap(&map_x);
        ptx::prefetch_tensormap(&map_w);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&ctl->tmem_base, TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    ptx::cta_sync();
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0, wfree_par = 0;
            int cur_n = -1;
            const uint64_t x_policy = l2_policy_evict_last();      // x is re-read once per panel: keep it in L2
            for (int t = t_begin; t < t_end && !*abort_flag; ++t) {
                const int n_tile = t / tiles_m, m0 = (t % tiles_m) * BM;
                if (n_tile != cur_n) {
                    if (cur_n >= 0) {                                  // all MMAs that read the old panel are done
                        if (!wait_or_abort(&ctl->w_free, wfree_par, abort_flag)) break;
                        wfree_par ^= 1;
                    }
                    ptx::mbar_arrive_expect_tx(&ctl->w_full, (uint32_t)(p.kb * w_block));
                    for (int kb = 0; kb < p.kb; ++kb)
                        ptx::tma_load_2d(W_s + (size_t)kb * w_block, &map_w, &ctl->w_full, kb * BK, n_tile * p.bn);
                    cur_n = n_tile;
                }
                for (int kb = 0; kb < p.kb; ++kb) {
                    if (!wait_or_abort(&ctl->a_empty[stage], phase ^ 1, abort_flag)) break;
                    ptx::mbar_arrive_expect_tx(&ctl->a_full[stage], A_BYTES);
                    tma_load_2d_hint(ring + (size_t)stage * A_BYTES, &map_x, &ctl->a_full[stage], kb * BK, m0, x_policy);
                    if (++stage == p.stages) { stage = 0; phase ^= 1; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = ptx::idesc_i8(BM, p.bn);
            int stage = 0; uint32_t phase = 0, wfull_par = 0;
            int cur_n = -1, it = 0;
            for (int t = t_begin; t < t_end && !*abort_flag; ++t, ++it) {
                const int n_tile = t / tiles_m;
                if (n_tile != cur_n) {
                    if (!wait_or_abort(&ctl->w_full, wfull_par, abort_flag)) break;
                    wfull_par ^= 1;
                    cur_n = n_tile;
                }
                const int buf = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1;
                if (!wait_or_abort(&ctl->tmem_empty[buf], acc_phase ^ 1, abort_flag)) break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * p.bn);
                bool ok = true;
                for (int kb = 0; kb < p.kb; ++kb) {
                    if (!wait_or_abort(&ctl->a_full[stage], phase, abort_flag)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint64_t a_desc = ptx::smem_desc_k_sw128(ptx::smem_u32(ring + (size_t)stage * A_BYTES));
                    const uint64_t b_desc = ptx::smem_desc_k_sw128(ptx::smem_u32(W_s + (size_t)kb * w_block));
#pragma unroll
                    for (int k = 0; k < BK / 32; ++k)     // 32 int8 = 32 bytes = 2 descriptor units along K
                        ptx::mma_i8_ss(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0);
                    ptx::mma_commit(&ctl->a_empty[stage]);  // frees the ring stage once these MMAs are done
                    if (++stage == p.stages) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                ptx::mma_commit(&ctl->tmem_full[buf]);
                if (t + 1 < t_end && (t + 1) / tiles_m != cur_n) ptx::mma_commit(&ctl->w_free);
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue ----------------
        const int e = warp - 2;
        const int quarter = warp & 3;                    // TMEM lanes this warp may read: 32 * (warp % 4)
        const int cgrp = e >> 2;                         // this warp takes the adjacent 32-column chunks 2 cgrp, 2 cgrp + 1:
                                                         // each thread then writes whole 128-byte lines of its row
        int32_t *bias = bias_s + e * BIAS_PER_WARP;
        const int n_chunks = p.bn >> 5;
        const int c0 = 2 * cgrp, c1 = 2 * cgrp + 1;
        const bool has0 = c0 < n_chunks, has1 = c1 < n_chunks;
        const bool wide_ok = (p.N % 16) == 0;            // every row starts on a 32-byte boundary
        int it = 0, cur_n0 = -1;
        const uint64_t st_policy = l2_policy_evict_first();        // the output is written once and read much later
        for (int t = t_begin; t < t_end; ++t, ++it) {
            const int buf = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1;
            const int n0 = (t / tiles_m) * p.bn, m0 = (t % tiles_m) * BM;
            if (n0 != cur_n0) {                          // the folded bias changes only with the panel
                __syncwarp();
                const int na = n0 + c0 * 32 + lane, nb = n0 + c1 * 32 + lane;
                bias[lane] = (has0 && na < p.N) ? p.bx[na] : 0;
                bias[32 + lane] = (has1 && nb < p.N) ? p.bx[nb] : 0;
                cur_n0 = n0;
                __syncwarp();
            }
            if (!__all_sync(0xffffffffu, wait_or_abort(&ctl->tmem_full[buf], acc_phase, abort_flag))) break;
            ptx::tc_fence_after();
            const int row = m0 + quarter * 32 + lane;
            const uint32_t tbase = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * p.bn);
            // the warp's 64 columns in four pieces of 16; the next piece's TMEM load is in flight while one is processed
            uint32_t ra[16], rb[16];
            const int np = (has0 ? 2 : 0) + (has1 ? 2 : 0);
            const uint32_t tcol = tbase + (uint32_t)(c0 * 32);
            const int n_base = n0 + c0 * 32;
            int16_t *dst_row = p.out + (size_t)row * p.N + n_base;
            const bool row_ok = row < p.M;
            // the gates' scales in the order of this warp's columns (with three gates the first column's gate varies)
            FastScale fs[4];
            Scale sc[4];
            if (G == 4) {
#pragma unroll
                for (int k = 0; k < 4; ++k) { fs[k] = p.fs[k]; sc[k] = p.sc[k]; }
            } else {
                const int first = n_base % 3;
#pragma unroll
                for (int k = 0; k < 3; ++k) {
                    const int g = first + k >= 3 ? first + k - 3 : first + k;
                    fs[k] = g == 0 ? p.fs[0] : g == 1 ? p.fs[1] : p.fs[2];
                    sc[k] = g == 0 ? p.sc[0] : g == 1 ? p.sc[1] : p.sc[2];
                }
                fs[3] = fs[0]; sc[3] = sc[0];
            }
            if (np > 0) ptx::tmem_ld_32x16(tcol, ra);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (i >= np) break;                                  // warp-uniform
                ptx::tmem_ld_wait();
                __syncwarp();
                if (i + 1 < np) {
                    if (i & 1) ptx::tmem_ld_32x16(tcol + (uint32_t)(16 * (i + 1)), ra);
                    else ptx::tmem_ld_32x16(tcol + (uint32_t)(16 * (i + 1)), rb);
                }
                const int n_valid = p.N - (n_base + 16 * i);
                if (row_ok && n_valid > 0) {
                    if (i & 1) epilogue_piece<G, GENERIC>(rb, bias + 16 * i, fs, sc, i, dst_row + 16 * i, n_valid, wide_ok, st_policy);
                    else epilogue_piece<G, GENERIC>(ra, bias + 16 * i, fs, sc, i, dst_row + 16 * i, n_valid, wide_ok, st_policy);
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ctl->tmem_empty[buf]);
        }
    }

    // ---------------- teardown ----------------
    ptx::cta_sync();
    if (*abort_flag) {
        // a wait ran out: give copies in flight time to land, then report
        for (int i = 0; i < 200; ++i) __nanosleep(500);
        if (threadIdx.x == 0) atomicExch(p.status, 1);
    }
    ptx::cta_sync();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

size_t smem_bytes(int bn, int kb, int stages)
{
    return 1024 + (size_t)kb * bn * BK + (size_t)stages * A_BYTES + EPI_WARPS * BIAS_PER_WARP * sizeof(int32_t) +
           sizeof(SharedCtl) + 64;
}

int ring_stages(int bn, int kb, int max_smem)
{
    int stages = MAX_STAGES;
    while (stages >= 2 && smem_bytes(bn, kb, stages) > (size_t)max_smem) --stages;
    return stages;
}

// How a launch of `rows` rows is cut: tiles per CTA and, if one panel per CTA costs no more tiles per CTA than equal
// contiguous ranges, the number of m-tile ranges (else 0).
struct TilePlan { int per_cta, m_ranges, grid; };

TilePlan plan_tiles(long long rows, int N, int bn, int sm_count)
{
    const int tiles_m = (int)((rows + BM - 1) / BM), tiles_n = (N + bn - 1) / bn;
    const long long tiles = (long long)tiles_m * tiles_n;
    TilePlan pl;
    pl.grid = tiles < sm_count ? (int)tiles : sm_count;
    pl.per_cta = pl.grid > 0 ? (int)((tiles + pl.grid - 1) / pl.grid) : 0;
    pl.m_ranges = 0;
    int ranges = sm_count / tiles_n;
    if (ranges > tiles_m) ranges = tiles_m;
    if (ranges > 0) {
        const int per = (tiles_m + ranges - 1) / ranges;
        ranges = (tiles_m + per - 1) / per;                  // drop ranges that would be empty
        if (per <= pl.per_cta) { pl.m_ranges = ranges; pl.grid = ranges * tiles_n; pl.per_cta = per; }
    }
    return pl;
}

// Panel width for launches of about `rows` rows.  A tile costs the larger of the epilogue (about 14.3 ns per column)
// and of streaming the x tile from L2 (128 rows x K bytes at about 29 GB/s per SM), a tenth more when the ring is
// too shallow to hold a whole x tile (the MMA issuer then waits on copies); all three figures were measured on
// B200.  Take the width, among those whose panel fits in shared memory, with the least tile time x tiles per CTA.
int panel_width(int K, int N, long long rows, int sm_count, int max_smem)
{
    const int kb = (K + BK - 1) / BK;
    int bn = (W_BYTES_MAX / (kb * BK)) / 32 * 32;
    bn = bn > 256 ? 256 : bn;
    if (rows <= 0) return bn;
    int best = bn;
    double best_cost = 1e30;
    for (int w = bn; w >= 32; w -= 32) {
        const int stages = ring_stages(w, kb, max_smem);
        if (stages < 2) continue;
        const double epilogue_ns = 14.3 * w, stream_ns = 128.0 * (kb * BK) / 29.0;
        const double tile_ns = (epilogue_ns > stream_ns ? epilogue_ns : stream_ns) * (stages < kb ? 1.1 : 1.0);
        const double cost = tile_ns * plan_tiles(rows, N, w, sm_count).per_cta;
        if (cost < best_cost) { best_cost = cost; best = w; }
    }
    return best;
}

}  // namespace

int debug_projection_plan(long long rows_hint, long long rows, int N, int K, int sm_count, int max_smem, int *out5)
{
    if (!out5 || rows_hint <= 0 || rows <= 0 || rows > rows_hint || N <= 0 || K <= 0 || sm_count <= 0 || max_smem <= 0)
        return QLSTM_ERR_ARG;
    const int kb = (K + BK - 1) / BK;
    const int bn = panel_width(K, N, rows_hint, sm_count, max_smem);
    const int stages = bn >= 32 ? ring_stages(bn, kb, max_smem) : 0;
    if (bn < 32 || stages < 2) return QLSTM_ERR_DIM;         // no resident panel for this K: the simple kernel runs
    const TilePlan pl = plan_tiles(rows, N, bn, sm_count);
    out5[0] = bn; out5[1] = stages; out5[2] = pl.per_cta; out5[3] = pl.m_ranges; out5[4] = pl.grid;
    return smem_bytes(bn, kb, stages) <= (size_t)max_smem ? QLSTM_OK : QLSTM_ERR_DIM;
}

bool fast_projection_supported(const FastLayer &f, const LayerParams &p)
{
    return f.proj_ok && (p.I % 16 == 0) && (p.N % 8 == 0);
}

int fast_projection_init(FastLayer &f, const LayerParams &p)
{
    f.proj_ok = false;
    if (p.I % 16 != 0 || p.N % 8 != 0) return 0;
    int dev = 0, max_smem = 0, sm_count = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
    const int bn = panel_width(p.I, p.N, f.proj_rows_hint, sm_count, max_smem);
    if (bn < 32) return 0;                                   // K too large for a resident panel
    const int kb = (p.I + BK - 1) / BK;
    const int stages = ring_stages(bn, kb, max_smem);
    if (stages < 2) return 0;
    f.proj_bn = bn;
    f.proj_stages = stages;
    if (!make_tensor_map_i8(&f.map_W, p.W, (uint64_t)p.N, (uint64_t)p.I, (uint32_t)bn, BK)) return 0;
    if (cudaFuncSetAttribute(k_projection_sm100<4, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess ||
        cudaFuncSetAttribute(k_projection_sm100<4, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess ||
        cudaFuncSetAttribute(k_projection_sm100<3, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess ||
        cudaFuncSetAttribute(k_projection_sm100<3, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess)
        return 0;
    f.proj_ok = true;
    return 0;
}

cudaError_t launch_projection_fast(const FastLayer &f, const LayerParams &p, const int8_t *x, int rows, int16_t *X,
                                   int sm_count, int *status, cudaStream_t st)
{
    CUtensorMap map_x;
    if (!make_tensor_map_i8(&map_x, x, (uint64_t)rows, (uint64_t)p.I, BM, BK)) return cudaErrorInvalidValue;
    ProjParams pp;
    pp.M = rows; pp.N = p.N; pp.K = p.I; pp.G = p.G;
    pp.bn = f.proj_bn; pp.kb = (p.I + BK - 1) / BK; pp.stages = f.proj_stages;
    pp.bx = p.bx; pp.out = X; pp.status = status; pp.generic = 0;
    for (int g = 0; g < 4; ++g) {
        Scale s = g < p.G ? p.eff_x[g] : Scale{0, 0};
        pp.sc[g] = s;
        if (s.shift > 0) pp.generic = 1;
        pp.fs[g] = make_fast_scale(s);
    }
    const TilePlan pl = plan_tiles(rows, p.N, pp.bn, sm_count);
    const int grid = pl.grid;
    pp.m_ranges = pl.m_ranges;
    const size_t smem = smem_bytes(pp.bn, pp.kb, pp.stages);
    if (p.G == 4) {
        if (pp.generic) k_projection_sm100<4, true><<<grid, THREADS, smem, st>>>(map_x, f.map_W, pp);
        else k_projection_sm100<4, false><<<grid, THREADS, smem, st>>>(map_x, f.map_W, pp);
    } else {
        if (pp.generic) k_projection_sm100<3, true><<<grid, THREADS, smem, st>>>(map_x, f.map_W, pp);
        else k_projection_sm100<3, false><<<grid, THREADS, smem, st>>>(map_x, f.map_W, pp);
    }
    return cudaGetLastError();
}

}  // namespace ql
