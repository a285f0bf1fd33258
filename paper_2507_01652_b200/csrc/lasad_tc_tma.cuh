// Host-side helper shared by the tensor-core prefill kernels: the TMA descriptor of one
// [B,T,H,64] bf16 tensor, tiled in chunks of 128 tokens of one head.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

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
inline bool encode_chunk_map_uncached(CUtensorMap* map, const void* base, int B, int T, int H, const long long* strides)
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

// The same through a small per-thread cache: a descriptor depends on nothing but the arguments
// below, and callers come back with the same tensors call after call (a layer's buffers, the
// slots of a host pipeline), so the driver call is made once per tensor, not once per launch.
inline bool encode_chunk_map(CUtensorMap* map, const void* base, int B, int T, int H, const long long* strides)
{
    struct Entry {
        const void* base;
        int B, T, H;
        long long s[3];
        bool valid;
        CUtensorMap map;
    };
    constexpr int kEntries = 32;
    thread_local Entry cache[kEntries];
    const unsigned long long x = (unsigned long long)reinterpret_cast<uintptr_t>(base);
    Entry& e = cache[((x >> 8) ^ (x >> 20) ^ (unsigned)T) % kEntries];
    if (e.valid && e.base == base && e.B == B && e.T == T && e.H == H && e.s[0] == strides[0] && e.s[1] == strides[1] &&
        e.s[2] == strides[2]) {
        *map = e.map;
        return true;
    }
    if (!encode_chunk_map_uncached(map, base, B, T, H, strides)) return false;
    e.base = base; e.B = B; e.T = T; e.H = H;
    e.s[0] = strides[0]; e.s[1] = strides[1]; e.s[2] = strides[2];
    e.map = *map;
    e.valid = true;
    return true;
}

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per device and kernel instead of once per
// launch.  `done` is the call site's own flag array.
template <typename Kernel>
inline cudaError_t allow_dynamic_smem(Kernel kernel, size_t bytes, bool (&done)[64])
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
    return e;
}

}  // namespace tcx
}  // namespace lasad
