// Host-side construction of TMA tensor maps.  The driver entry point is looked up through
// the runtime so that the library does not link against libcuda (it must load on machines
// without a driver, where only argument checks run).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace salad {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_tiled() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) ==
                cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Map over a bf16 tensor [outer, rows, d] (d fastest, contiguous).  One box is
// [1, box_rows, 64] elements = box_rows x 128 bytes, written to shared memory with the
// 128-byte swizzle.  Rows past `rows` read as zero and are not written by stores, so a
// ragged last block never touches the next head.
inline bool make_tmap_bf16_3d(CUtensorMap* out, const void* base, int d, int64_t rows,
                              int64_t outer, int box_rows) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return false;
    cuuint64_t dims[3] = {cuuint64_t(d), cuuint64_t(rows), cuuint64_t(outer)};
    cuuint64_t strides[2] = {cuuint64_t(d) * 2, cuuint64_t(d) * 2 * cuuint64_t(rows)};
    cuuint32_t box[3] = {64, cuuint32_t(box_rows), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims,
                     strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Map over the same bf16 tensor [outer, N, d] whose N = T * S tokens are numbered with time slowest
// (n = t * S + s), seen as [outer, S, T, d]: a box of [1, box_s, T, 64] elements is box_s * T rows of 128
// bytes in shared memory, row s_local * T + t -- the tokens of box_s spatial positions in the order that
// groups tokens by spatial position (Appendix A.1), without the tensor being re-ordered in memory.
// Spatial positions past S read as zero and are not written by stores.
inline bool make_tmap_bf16_4d_by_position(CUtensorMap* out, const void* base, int d, int T, int64_t S,
                                          int64_t outer, int box_s) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return false;
    cuuint64_t dims[4] = {cuuint64_t(d), cuuint64_t(T), cuuint64_t(S), cuuint64_t(outer)};
    cuuint64_t strides[3] = {cuuint64_t(S) * d * 2, cuuint64_t(d) * 2, cuuint64_t(T) * cuuint64_t(S) * d * 2};
    cuuint32_t box[4] = {64, cuuint32_t(T), cuuint32_t(box_s), 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims,
                     strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Map over an fp16 matrix [rows, cols] (cols fastest, contiguous; cols <= 256).  One box is
// [box_rows, cols], written to shared memory row after row without swizzle.  Rows past `rows`
// read as zero.
inline bool make_tmap_f16_rows(CUtensorMap* out, const void* base, int cols, int64_t rows, int box_rows) {
    EncodeTiledFn enc = get_encode_tiled();
    if (!enc) return false;
    cuuint64_t dims[3] = {cuuint64_t(cols), cuuint64_t(rows), 1};
    cuuint64_t strides[2] = {cuuint64_t(cols) * 2, cuuint64_t(cols) * 2 * cuuint64_t(rows)};
    cuuint32_t box[3] = {cuuint32_t(cols), cuuint32_t(box_rows), 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(base), dims,
                     strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace salad
