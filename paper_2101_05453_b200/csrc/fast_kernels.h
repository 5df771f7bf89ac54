// Interface between the host API and the sm_100a fast kernels (tensor-core input projection,
// persistent recurrent kernel).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <vector>

#include "act_table.cuh"
#include "qlstm_internal.h"

namespace ql {

// Device scratch of the persistent recurrent kernel, shared by all layers of a handle.
struct FastScratch {
    int Bpad = 0;                // max batch rounded up to 128: rows of the MMA operands
    int sm_count = 0;
    int8_t *hbuf = nullptr;      // [2][Bpad x max O]  h^{t-1} / h^t, the recurrent matmul's A operand (tiled k-block image,
                                 //                    plain rows at small batch)
    int8_t *mbuf = nullptr;      // [Bpad x max C]     hidden state m, the projection's A operand (same layouts)
    int32_t *pre = nullptr;      // [max B][max N]    layer norm: gate sums between the matmul and elementwise phases
                                 //                   (int16 values, or int32 X+H when a peephole follows)
    unsigned *bar = nullptr;     // [0] grid-barrier counter, [1] abort word
    size_t hbuf_bytes = 0, mbuf_bytes = 0;
};

struct FastLayer {
    bool proj_ok = false;        // tensor-core projection usable for this layer
    CUtensorMap map_W;           // W [N][I] int8, K-major, 128B swizzle, box = one k-block of the resident panel
    int proj_bn = 0;             // panel width (rows of W resident in shared memory)
    long long proj_rows_hint = 0; // rows (max_T * max_B) the panel width is tuned for; set before fast_layer_init
    int proj_stages = 0;         // depth of the x ring
    // persistent recurrent kernel plan
    bool rec_ok = false;
    int grid = 0;                // CTAs of the cooperative launch (one per SM)
    int cpc = 0;                 // cells per CTA in the matmul phase
    int n_cta_a = 0;             // CTAs that own cells
    int nc_pad = 0;              // UMMA N of the recurrent matmul (multiple of 16)
    int pn = 0, npn = 0;         // projection: N-slice width and number of N slices
    int kb_h = 0, kb_c = 0;      // 128-byte k-blocks of the recurrent / projection matmul
    int stages = 0;              // ring stages (power of two)
    int n_issue_c = 1;           // projection MMA issuers, each with its own partial accumulator
    size_t smem = 0;
    CUtensorMap map_R, map_Wp;   // resident weight slices; the streamed operands h, m use plain bulk copies
    // memoised sigmoid / tanh of the elementwise phase (act_table.cuh): device blob and its layout; null: arithmetic path
    uint8_t *act_tab = nullptr;
    ActTabLayout act_lay = {0, 0, 0, 0, 0, 0, 0};
    bool dbg_no_tables = false;  // test hook: keep the arithmetic path although the tables exist
    bool dbg_general_kernel = false;   // test hook: the instantiation that accepts scales with a left shift
    // test hook: make every grid barrier expect `dbg_barrier_extra` arrivals that never come, with a short wait limit
    unsigned dbg_barrier_extra = 0;
    unsigned long long dbg_spin_limit_ns = 0;
};

int fast_scratch_init(FastScratch &s, int max_B, int maxC, int maxO, int maxN, int sm_count);
void fast_scratch_destroy(FastScratch &s);

int fast_layer_init(FastLayer &f, const LayerParams &p, const FastScratch &s, int max_T, int max_B);
void fast_layer_destroy(FastLayer &f);
int fast_projection_init(FastLayer &f, const LayerParams &p);
int fast_recurrent_init(FastLayer &f, const LayerParams &p, const FastScratch &s, int max_B);

bool fast_projection_supported(const FastLayer &f, const LayerParams &p);
cudaError_t launch_projection_fast(const FastLayer &f, const LayerParams &p, const int8_t *x, int rows, int16_t *X,
                                   int sm_count, int *status, cudaStream_t st);

bool fast_recurrent_supported(const FastLayer &f, const LayerParams &p, int B);
// h / c are the caller's state (B rows); y is [T][B][O].  Batches up to small_batch_max (at most 16) run the matmuls
// as dp4a mat-vecs.  Returns a qlstm_error.
int launch_recurrent_fast(const FastLayer &f, const LayerParams &p, const FastScratch &s, const int16_t *X, int T, int B,
                          int8_t *h, int16_t *c, int8_t *y, int *status, unsigned long long *phase_ns, int small_batch_max,
                          cudaStream_t st, int *launches);

// Host logic of the recurrent kernel's operand ring, for tests: fills out[14] = n_own, n_max, n_chunks[4], cnt[4],
// uses[4] of the plan for `stages` ring stages and `n_own` issuers (see RingPlan in recurrent_sm100.cu).
// ---- whole-stack kernel for small batches (stack_small_sm100.cu): all layers and steps in one cooperative launch,
// one group of blocks per layer, layers running as a wavefront; also the path of one-step (streaming) calls.
constexpr int STACK_SMALL_MAX_B = 16;
struct StackSmall;
int stack_small_create(const std::vector<const LayerParams *> &layers, int max_T, int max_B, int sm_count, StackSmall **out);
void stack_small_destroy(StackSmall *s);
bool stack_small_supported(const StackSmall *s, int T, int B);
bool stack_small_preferred(const StackSmall *s, int T, int B);     // supported and, by measurement, the faster path
// schedule: 0 automatic, 1 wavefront (one group of blocks per layer), 2 sequential (every layer on all blocks).
// The kernel clears the status word itself.
int launch_stack_small(StackSmall *s, const int8_t *x, int T, int B, int8_t *h, int16_t *c, int8_t *y, int *status,
                       int schedule, cudaStream_t st);
void stack_small_debug_timeout(StackSmall *s, unsigned missing_arrivals, unsigned long long limit_ns);
int stack_small_groups(const StackSmall *s, int *blocks_per_layer);     // layers, and the blocks each layer's group has

int debug_ring_plan(int stages, int n_own, int contig, int per, int n_total, int *out);
int debug_projection_plan(long long rows_hint, long long rows, int N, int K, int sm_count, int max_smem, int *out5);

}  // namespace ql
