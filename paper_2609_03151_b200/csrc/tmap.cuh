// Host-side construction of TMA tensor maps without linking libcuda: the driver's encoder
// is looked up through the runtime (cudaGetDriverEntryPoint) on first use.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "common.cuh"

namespace tmap {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encoder() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// bf16 tensor [rows][heads][D] (D fastest) seen as 3-D (D, heads, rows); box = 64 x 1 x box_rows
// elements with the 128-byte swizzle (each box row is one 128-byte line).
// The encoder costs a few microseconds per map and a launch needs three maps per rank; callers that launch again and
// again on the same buffers (a layer called every step, the pieces of the host-buffer entry) get them from a small
// per-thread memo keyed by every argument (host memory only; a map is a pure function of its arguments).
struct MemoEntry {
    const void *base = nullptr;
    uint64_t rows = 0, heads = 0, D = 0;
    uint32_t box_rows = 0;
    CUtensorMap map;
};
constexpr int kMemoSlots = 256;

inline int encode_rows_heads_d_uncached(CUtensorMap *out, const void *base, uint64_t rows, uint64_t heads, uint64_t D,
                                        uint32_t box_rows);

inline int encode_rows_heads_d(CUtensorMap *out, const void *base, uint64_t rows, uint64_t heads, uint64_t D,
                               uint32_t box_rows) {
    static thread_local MemoEntry memo[kMemoSlots];
    const uint64_t h = ((uint64_t)(uintptr_t)base >> 8) * 0x9E3779B97F4A7C15ull + rows * 31 + heads * 7 + D + box_rows;
    MemoEntry &e = memo[(h >> 32) % kMemoSlots];
    if (e.base == base && e.rows == rows && e.heads == heads && e.D == D && e.box_rows == box_rows) {
        *out = e.map;
        return BASP_OK;
    }
    const int rc = encode_rows_heads_d_uncached(out, base, rows, heads, D, box_rows);
    if (rc == BASP_OK) { e.base = base; e.rows = rows; e.heads = heads; e.D = D; e.box_rows = box_rows; e.map = *out; }
    return rc;
}

inline int encode_rows_heads_d_uncached(CUtensorMap *out, const void *base, uint64_t rows, uint64_t heads, uint64_t D,
                                        uint32_t box_rows) {
    EncodeTiledFn fn = encoder();
    if (!fn) {
        basp_set_cuda_error("cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)", -1, "driver entry point not found");
        return BASP_ERR_CUDA;
    }
    cuuint64_t dims[3] = {D, heads, rows};
    cuuint64_t strides[2] = {D * 2, heads * D * 2};
    cuuint32_t box[3] = {64, 1, box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        basp_set_cuda_error("cuTensorMapEncodeTiled", (int)r, "tensor map encoding failed");
        return BASP_ERR_CUDA;
    }
    return BASP_OK;
}

// fp32 tensor [rows][heads][D] seen as 3-D (D, heads, rows); box = 32 x 1 x box_rows floats (128-byte
// lines) with the 128-byte swizzle: the shape of one warp's share of an accumulator tile.
inline int encode_f32_rows_heads_d(CUtensorMap *out, const void *base, uint64_t rows, uint64_t heads, uint64_t D,
                                   uint32_t box_rows) {
    EncodeTiledFn fn = encoder();
    if (!fn) {
        basp_set_cuda_error("cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)", -1, "driver entry point not found");
        return BASP_ERR_CUDA;
    }
    cuuint64_t dims[3] = {D, heads, rows};
    cuuint64_t strides[2] = {D * 4, heads * D * 4};
    cuuint32_t box[3] = {32, 1, box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        basp_set_cuda_error("cuTensorMapEncodeTiled(f32)", (int)r, "tensor map encoding failed");
        return BASP_ERR_CUDA;
    }
    return BASP_OK;
}

}  // namespace tmap
