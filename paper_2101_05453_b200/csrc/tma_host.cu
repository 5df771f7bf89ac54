#include "tma_host.h"

#include <cudaTypedefs.h>

namespace ql {

static PFN_cuTensorMapEncodeTiled_v12000 encode_fn()
{
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (PFN_cuTensorMapEncodeTiled_v12000)p;
    }
    return fn;
}

static bool encode(CUtensorMap *map, CUtensorMapDataType dt, size_t esize, const void *base, uint64_t rows,
                   uint64_t cols, uint32_t box_rows, uint32_t box_cols, CUtensorMapSwizzle sw)
{
    auto fn = encode_fn();
    if (!fn) return false;
    if (((uintptr_t)base & 15) || ((cols * esize) & 15)) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * esize};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, dt, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool make_tensor_map_i8(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                        uint32_t box_cols)
{
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, base, rows, cols, box_rows, box_cols, CU_TENSOR_MAP_SWIZZLE_128B);
}

bool make_tensor_map_i16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                         uint32_t box_cols)
{
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, base, rows, cols, box_rows, box_cols, CU_TENSOR_MAP_SWIZZLE_NONE);
}

}  // namespace ql
