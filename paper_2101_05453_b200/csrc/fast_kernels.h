// Interface between the host API and the sm_100a fast kernels (tensor-core input projection,
// persistent recurrent kernel).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "qlstm_internal.h"

namespace ql {

struct FastLayer {
    bool proj_ok = false;        // tensor-core projection usable for this layer
    bool rec_ok = false;         // persistent recurrent kernel usable for this layer
    CUtensorMap map_W;           // W [N][I] int8, K-major, 128B swizzle
    int proj_block_n = 0;
    // persistent kernel tiling
    int cells_per_cta = 0, n_cta = 0, proj_cols_per_cta = 0;
    CUtensorMap map_R, map_Wproj;
    void *dev_aux = nullptr;
};

struct FastScratch {
    int persistent_blocks = 0;
    int8_t *hbuf = nullptr;      // padded double-buffered h operand
    int8_t *mbuf = nullptr;      // padded m operand
    long long *ln_part = nullptr;
    unsigned *bar = nullptr;     // grid barrier words
    int max_B = 0;
};

int fast_layer_init(FastLayer &f, const LayerParams &p, int max_T, int max_B, int sm_count);
int fast_projection_init(FastLayer &f, const LayerParams &p);
void fast_layer_destroy(FastLayer &f);
int fast_scratch_init(FastScratch &s, int max_B, int maxC, int maxO, int maxN, int sm_count);
void fast_scratch_destroy(FastScratch &s);
int fast_persistent_blocks(const FastScratch &s);

bool fast_projection_supported(const FastLayer &f, const LayerParams &p);
cudaError_t launch_projection_fast(const FastLayer &f, const LayerParams &p, const int8_t *x, int rows, int16_t *X,
                                   int sm_count, int *status, cudaStream_t st);

bool fast_recurrent_supported(const FastLayer &f, const LayerParams &p, int B);
int launch_recurrent_fast(const FastLayer &f, const LayerParams &p, const FastScratch &s, const int16_t *X, int T, int B,
                          int8_t *h, int16_t *c, int8_t *y, int *status, cudaStream_t st, int *launches);

}  // namespace ql
