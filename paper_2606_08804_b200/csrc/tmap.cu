// Host side: tensor maps (TMA descriptors) of the bf16 tiles the tensor-core kernels copy, and the once-only
// shared-memory attribute of the kernels.
// Every map uses boxes of 64 elements (128 bytes) along the innermost dimension and the 128-byte
// swizzle, i.e. exactly the shared-memory operand layout described in sm100.cuh.
#include "internal.h"
#include "sm100.cuh"

#include <cudaTypedefs.h>

#include <mutex>

namespace qd {
namespace {

PFN_cuTensorMapEncodeTiled_v12000 encoder() {
    static PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess || !fn)
            return nullptr;
        encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
    }
    return encode;
}

}  // namespace

bool make_tmap_bf16_2d(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes,
                       uint32_t box_rows) {
    PFN_cuTensorMapEncodeTiled_v12000 encode = encoder();
    if (!encode) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool make_tmap_tokens(CUtensorMap* map, const void* base, int B, int T, int H, int D, uint32_t box_rows) {
    PFN_cuTensorMapEncodeTiled_v12000 encode = encoder();
    if (!encode) return false;
    const uint64_t cols = (uint64_t)H * D;
    cuuint64_t dims[3] = {cols, (uint64_t)T, (uint64_t)B};
    cuuint64_t strides[2] = {cols * 2, (uint64_t)T * cols * 2};
    cuuint32_t box[3] = {64, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

cudaError_t set_max_smem_once(const void* kernel, size_t bytes) {
    // fixed table, no heap: the largest size set so far for each (kernel, device)
    struct Entry { const void* kernel; int dev; size_t bytes; };
    static std::mutex mu;
    static Entry table[128];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    Entry* slot = nullptr;
    for (Entry& t : table) {
        if (!t.kernel || (t.kernel == kernel && t.dev == dev)) { slot = &t; break; }
    }
    if (slot && slot->kernel && slot->bytes >= bytes) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess && slot) { slot->kernel = kernel; slot->dev = dev; slot->bytes = bytes; }
    return e;
}

}  // namespace qd
