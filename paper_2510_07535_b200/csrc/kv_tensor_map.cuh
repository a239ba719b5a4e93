// Host side: TMA tensor maps over the paged KV cache.
//
// The cache is bf16 (or fp16) [num_pages, Hkv, page_size, 128]; one (page, head) block is page_size rows of
// 256 bytes.  The tensor-core operands want each 128-key tile in shared memory as 8-key groups of
// two 1024-byte swizzle atoms: [key group][half of the head dimension][8 keys][64 elements], with
// the 128-byte swizzle.  One TMA box per (page, head) produces exactly that when the tensor is
// described in five dimensions ordered as the shared-memory image wants them:
//   dim0 = 64 elements of one half (contiguous), dim1 = 8 keys of a group (stride 256 B),
//   dim2 = the 2 halves (stride 128 B), dim3 = page_size/8 key groups (stride 2048 B),
//   dim4 = page * Hkv + head (stride page_size * 256 B).
// The innermost coordinate of every copy is 0, so the 16-byte start rule of TMA holds by construction.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace owl {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Looks the driver entry point up through the runtime (no link-time dependency on libcuda).
inline EncodeTiledFn load_encode_tiled() {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
        return nullptr;
    return reinterpret_cast<EncodeTiledFn>(fn);
}

// Returns 0 on success, else the CUresult of the encode call (or -1 if the entry point is missing).
inline int make_kv_tensor_map(EncodeTiledFn encode, CUtensorMap* map, const void* cache, long long num_pages,
                              int num_kv_heads, int page_size, bool fp16) {
    if (!encode) return -1;
    const cuuint64_t dims[5] = {64, 8, 2, (cuuint64_t)(page_size / 8), (cuuint64_t)(num_pages * num_kv_heads)};
    const cuuint64_t strides[4] = {256, 128, 2048, (cuuint64_t)page_size * 256};   // bytes, dims 1..4
    const cuuint32_t box[5] = {64, 8, 2, (cuuint32_t)(page_size / 8), 1};
    const cuuint32_t elem_strides[5] = {1, 1, 1, 1, 1};
    CUresult r = encode(map, fp16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(cache), dims, strides, box,
                        elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return (int)r;
}

}  // namespace owl
