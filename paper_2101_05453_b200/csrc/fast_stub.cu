// Placeholder until the sm_100a fast kernels land: reports every shape as unsupported.
#include "fast_kernels.h"
#include "../../include/qlstm.h"
namespace ql {
int fast_layer_init(FastLayer &f, const LayerParams &p, int, int, int) { return fast_projection_init(f, p); }
void fast_layer_destroy(FastLayer &) {}
int fast_scratch_init(FastScratch &, int, int, int, int, int) { return QLSTM_OK; }
void fast_scratch_destroy(FastScratch &) {}
int fast_persistent_blocks(const FastScratch &s) { return s.persistent_blocks; }
bool fast_recurrent_supported(const FastLayer &, const LayerParams &, int) { return false; }
int launch_recurrent_fast(const FastLayer &, const LayerParams &, const FastScratch &, const int16_t *, int, int, int8_t *, int16_t *, int8_t *, int *, cudaStream_t, int *) { return QLSTM_ERR_DIM; }
}
