// Host-side helper shared by the tensor-core prefill kernels: the TMA descriptor of one
// [B,T,H,64] bf16 tensor, tiled in chunks of 128 tokens of one head.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

namespace lasad {
namespace tcx {

// cuTensorMapEncodeTiled, fetched through the runtime so that the library does not link libcuda.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// [B,T,H,64] bf16 with element strides (b,t,h) -> 4-D map (d, h, t, b); box = 128 tokens of one
// head, rows of 128 bytes with the 128-byte swizzle; rows past T read as zeros and are not stored.
inline bool encode_chunk_map(CUtensorMap* map, const void* base, int B, int T, int H, const long long* strides)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    auto bytes = [](long long elems) { return (cuuint64_t)(elems > 0 ? elems * 2 : 128); };
    const cuuint64_t dims[4] = {64u, (cuuint64_t)H, (cuuint64_t)T, (cuuint64_t)B};
    const cuuint64_t gstr[3] = {bytes(strides[2]), bytes(strides[1]), bytes(strides[0])};
    const cuuint32_t box[4] = {64u, 1u, 128u, 1u};
    const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, gstr, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tcx
}  // namespace lasad
