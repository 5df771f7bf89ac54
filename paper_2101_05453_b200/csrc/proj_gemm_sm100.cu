// Batched input projection on the 5th-generation tensor cores (Section 3.2.4, first rescale term):
//
//   X[r][n] = sat16( rescale( sum_j W[n][j] * x[r][j] + bx[n], eff_x[gate(n)] ) ),   r < rows, n < N = C*G
//
// int8 x int8 -> int32 dense contraction, so it runs as tcgen05.mma kind::i8 with the int32
// accumulator in tensor memory.  The rescale to int16 is fused into the epilogue: writing int32
// accumulators would double the HBM traffic of a kernel whose output already costs as much time
// as its math (K is only 512-1024).
//
// One persistent CTA per SM, warp specialised:
//   warp 0      TMA producer: x tile [128 x 128 B] and W tile [256 x 128 B] per k-block, 4-stage ring
//   warp 1      MMA issuer:   4 x (M128 N256 K32) per k-block into one of two 256-column TMEM buffers
//   warps 2..9  epilogue:     tcgen05.ld -> + folded bias -> fixed-point rescale -> sat16 -> 16-byte stores,
//                             overlapping the next tile's MMAs through the second TMEM buffer
// No cluster launch and no multicast.
#include "fast_kernels.h"
#include "sm100_ptx.cuh"
#include "tma_host.h"

namespace ql {

namespace {

constexpr int BM = 128, BN = 256, BK = 128, STAGES = 4, EPI_WARPS = 8;
constexpr int A_BYTES = BM * BK, B_BYTES = BN * BK, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int THREADS = 32 * (2 + EPI_WARPS);
constexpr int TMEM_COLS = 512;
constexpr size_t SMEM_BYTES = 1024 /*align slack*/ + (size_t)STAGES * STAGE_BYTES + EPI_WARPS * 128 * sizeof(int32_t) + 256;

struct ProjParams {
    int M, N, K, G;
    const int32_t *bx;
    int16_t *out;
    FastScale fs[4];
    Scale sc[4];
    int generic;        // some gate has a positive shift: use the generic rescale
    int *status;
};

struct SharedCtl {
    uint64_t full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ bool wait_or_abort(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    for (uint32_t i = 0; i < (1u << 20); ++i) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

template <int G>
__device__ __forceinline__ void epilogue_chunk(const uint32_t (&r)[32], const int32_t *bias, const ProjParams &p,
                                               int n_first, int16_t *dst, int n_valid)
{
    // column j of this chunk is global column n_first + j; its gate slot is (n_first + j) % G
    uint32_t packed[16];
    const int phase = n_first % G;
#pragma unroll
    for (int j = 0; j < 32; j += 2) {
        int32_t v0 = (int32_t)r[j] + bias[j], v1 = (int32_t)r[j + 1] + bias[j + 1];
        int g0, g1;
        if (G == 4) { g0 = j & 3; g1 = (j + 1) & 3; }
        else { g0 = (phase + j) % 3; g1 = (phase + j + 1) % 3; }
        int32_t y0, y1;
        if (p.generic) { y0 = mbqm(v0, p.sc[g0]); y1 = mbqm(v1, p.sc[g1]); }
        else { y0 = fast_rescale(v0, p.fs[g0]); y1 = fast_rescale(v1, p.fs[g1]); }
        packed[j >> 1] = ptx::pack_sat_s16(y0, y1);
    }
    if (n_valid >= 32) {
#pragma unroll
        for (int v = 0; v < 4; ++v)
            *reinterpret_cast<uint4 *>(dst + 8 * v) = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
    } else {
#pragma unroll
        for (int v = 0; v < 4; ++v)
            if (8 * v + 8 <= n_valid)
                *reinterpret_cast<uint4 *>(dst + 8 * v) = make_uint4(packed[4 * v], packed[4 * v + 1], packed[4 * v + 2], packed[4 * v + 3]);
    }
}

__global__ void __launch_bounds__(THREADS, 1)
k_projection_sm100(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, ProjParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *tiles = smem;
    int32_t *bias_s = (int32_t *)(smem + (size_t)STAGES * STAGE_BYTES);
    SharedCtl *ctl = (SharedCtl *)(bias_s + EPI_WARPS * 128);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles_m = (p.M + BM - 1) / BM, tiles_n = (p.N + BN - 1) / BN;
    const int n_tiles = tiles_m * tiles_n, k_blocks = (p.K + BK - 1) / BK;
    volatile int *abort_flag = &ctl->abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(&ctl->full[s], 1); ptx::mbar_init(&ctl->empty[s], 1); }
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
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x) {
                const int m0 = (t / tiles_n) * BM, n0 = (t % tiles_n) * BN;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!wait_or_abort(&ctl->empty[stage], phase ^ 1, abort_flag)) break;
                    uint8_t *a = tiles + (size_t)stage * STAGE_BYTES, *b = a + A_BYTES;
                    ptx::mbar_arrive_expect_tx(&ctl->full[stage], STAGE_BYTES);
                    ptx::tma_load_2d(a, &map_x, &ctl->full[stage], kb * BK, m0);
                    ptx::tma_load_2d(b, &map_w, &ctl->full[stage], kb * BK, n0);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t IDESC = ptx::idesc_i8(BM, BN);
            int stage = 0; uint32_t phase = 0;
            int it = 0;
            for (int t = blockIdx.x; t < n_tiles && !*abort_flag; t += gridDim.x, ++it) {
                const int buf = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1;
                if (!wait_or_abort(&ctl->tmem_empty[buf], acc_phase ^ 1, abort_flag)) break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)buf * BN;
                bool ok = true;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!wait_or_abort(&ctl->full[stage], phase, abort_flag)) { ok = false; break; }
                    ptx::tc_fence_after();
                    const uint32_t a_addr = ptx::smem_u32(tiles + (size_t)stage * STAGE_BYTES), b_addr = a_addr + A_BYTES;
                    const uint64_t a_desc = ptx::smem_desc_k_sw128(a_addr), b_desc = ptx::smem_desc_k_sw128(b_addr);
#pragma unroll
                    for (int k = 0; k < BK / 32; ++k)     // 32 int8 = 32 bytes = 2 descriptor units along K
                        ptx::mma_i8_ss(d_tmem, a_desc + 2 * k, b_desc + 2 * k, IDESC, (kb | k) != 0);
                    ptx::mma_commit(&ctl->empty[stage]);  // frees the smem stage once these MMAs are done
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (!ok) break;
                ptx::mma_commit(&ctl->tmem_full[buf]);
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue ----------------
        const int e = warp - 2;
        const int quarter = warp & 3;                    // TMEM lanes this warp may read: 32 * (warp % 4)
        const int half = e >> 2;                         // which 128 of the 256 columns
        int32_t *bias = bias_s + e * 128;                // this warp's 128 folded biases of the current tile
        int it = 0;
        for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++it) {
            const int buf = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1;
            const int m0 = (t / tiles_n) * BM, n0 = (t % tiles_n) * BN;
            __syncwarp();
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int n = n0 + half * 128 + i * 32 + lane;
                bias[i * 32 + lane] = n < p.N ? p.bx[n] : 0;
            }
            __syncwarp();
            if (!__all_sync(0xffffffffu, wait_or_abort(&ctl->tmem_full[buf], acc_phase, abort_flag))) break;
            ptx::tc_fence_after();
            const int row = m0 + quarter * 32 + lane;
#pragma unroll 1
            for (int ch = 0; ch < 4; ++ch) {
                const int col = half * 128 + ch * 32, cw = ch * 32;
                uint32_t r[32];
                __syncwarp();             // the TMEM load is warp-collective: reconverge after the per-row branch
                ptx::tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + col), r);
                ptx::tmem_ld_wait();
                const int n_first = n0 + col;
                int n_valid = p.N - n_first;
                if (row < p.M && n_valid > 0) {
                    int16_t *dst = p.out + (size_t)row * p.N + n_first;
                    if (p.G == 4) epilogue_chunk<4>(r, bias + cw, p, n_first, dst, n_valid);
                    else epilogue_chunk<3>(r, bias + cw, p, n_first, dst, n_valid);
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&ctl->tmem_empty[buf]);
        }
    }

    // ---------------- teardown ----------------
    __syncthreads();
    if (*abort_flag) {
        // a wait ran out: give copies in flight time to land, then report
        for (int i = 0; i < 200; ++i) __nanosleep(500);
        if (threadIdx.x == 0) atomicExch(p.status, 1);
    }
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace

bool fast_projection_supported(const FastLayer &f, const LayerParams &p)
{
    return f.proj_ok && (p.I % 16 == 0) && (p.N % 8 == 0);
}

int fast_projection_init(FastLayer &f, const LayerParams &p)
{
    f.proj_ok = false;
    if (p.I % 16 != 0 || p.N % 8 != 0) return 0;
    if (!make_tensor_map_i8(&f.map_W, p.W, (uint64_t)p.N, (uint64_t)p.I, BN, BK)) return 0;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(k_projection_sm100, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) != cudaSuccess)
            return 0;
        attr_set = true;
    }
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
    pp.bx = p.bx; pp.out = X; pp.status = status; pp.generic = 0;
    for (int g = 0; g < 4; ++g) {
        Scale s = g < p.G ? p.eff_x[g] : Scale{0, 0};
        pp.sc[g] = s;
        if (s.shift > 0) pp.generic = 1;
        int R = s.shift < 0 ? -s.shift : 0;
        pp.fs[g] = make_fast_scale(s);
        (void)R;
    }
    const int tiles = ((rows + BM - 1) / BM) * ((p.N + BN - 1) / BN);
    const int grid = tiles < sm_count ? tiles : sm_count;
    k_projection_sm100<<<grid, THREADS, SMEM_BYTES, st>>>(map_x, f.map_W, pp);
    return cudaGetLastError();
}

}  // namespace ql
