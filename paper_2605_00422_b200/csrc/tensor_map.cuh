// Host side of the TMA descriptors: cuTensorMapEncodeTiled is reached through the runtime's driver entry point query, so
// the library does not link against libcuda.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include "bwla_common.cuh"

namespace bwla {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// rank 2 or 3; dims/box innermost first; strides in bytes for dimensions 1..rank-1
inline int make_map(CUtensorMap* map, CUtensorMapDataType dt, int rank, const void* base, const uint64_t* dims,
                    const uint64_t* strides, const uint32_t* box, CUtensorMapSwizzle sw, CUtensorMapL2promotion promo) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return BWLA_ERR_CUDA;
    cuuint64_t d[3]; cuuint64_t s[2]; cuuint32_t b[3]; cuuint32_t estr[3] = {1, 1, 1};
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; }
    for (int i = 0; i + 1 < rank; ++i) s[i] = strides[i];
    CUresult r = fn(map, dt, (cuuint32_t)rank, const_cast<void*>(base), d, s, b, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                    promo, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return BWLA_ERR_CUDA; }
    return BWLA_OK;
}

}  // namespace bwla
