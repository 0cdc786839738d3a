// Host-side tensor-map (TMA descriptor) encoders shared by the convolution kernels' launchers.
// The driver entry points are looked up once through the runtime, so the library links against
// nothing but the static CUDA runtime.
#pragma once
#include <cuda.h>

#include <mutex>

#include "nm_internal.h"

namespace nmtm {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
using EncodeIm2colFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t, const cuuint32_t*,
                                    CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                    CUtensorMapFloatOOBfill);

struct Encoders {
    EncodeTiledFn tiled = nullptr;
    EncodeIm2colFn im2col = nullptr;
};

inline const Encoders& encoders()
{
    static Encoders enc;
    static std::once_flag once;
    std::call_once(once, [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            enc.tiled = reinterpret_cast<EncodeTiledFn>(f);
        f = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            enc.im2col = reinterpret_cast<EncodeIm2colFn>(f);
        (void)cudaGetLastError();
    });
    return enc;
}

inline bool available() { return encoders().tiled && encoders().im2col; }

// Activations as an im2col tensor map: NHWC seen as (C, W, H, N); the box is 32 channels x
// `pixels` output pixels; the base-pixel window runs from -pad to pad - (K - 1) * dil in each
// direction and is walked with the convolution stride.  128-byte swizzle.
inline bool encode_x_im2col(const ConvParams& p, int pixels, CUtensorMap* tm)
{
    const cuuint64_t dims[4] = {static_cast<cuuint64_t>(p.c_in), static_cast<cuuint64_t>(p.w),
                                static_cast<cuuint64_t>(p.h), static_cast<cuuint64_t>(p.batch)};
    const cuuint64_t strides[3] = {static_cast<cuuint64_t>(p.c_in) * 4, static_cast<cuuint64_t>(p.w) * p.c_in * 4,
                                   static_cast<cuuint64_t>(p.h) * p.w * p.c_in * 4};
    const int lower[2] = {-p.pad_w, -p.pad_h};
    const int upper[2] = {p.pad_w - (p.kw - 1) * p.dil_w, p.pad_h - (p.kh - 1) * p.dil_h};
    const cuuint32_t trav[4] = {1, static_cast<cuuint32_t>(p.stride_w), static_cast<cuuint32_t>(p.stride_h), 1};
    return encoders().im2col(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(p.x), dims, strides, lower,
                             upper, 32, static_cast<cuuint32_t>(pixels), trav, CU_TENSOR_MAP_INTERLEAVE_NONE,
                             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Geometry limits of the im2col map (corner offsets are 8-bit, traversal strides 3-bit).
inline bool im2col_geometry_ok(const ConvParams& p)
{
    if (p.pad_w > 127 || p.pad_h > 127) return false;
    if ((p.kw - 1) * p.dil_w - p.pad_w > 128 || (p.kh - 1) * p.dil_h - p.pad_h > 128) return false;
    if ((p.kw - 1) * p.dil_w > 65535 || (p.kh - 1) * p.dil_h > 65535) return false;
    if (p.stride_w > 8 || p.stride_h > 8) return false;
    return true;
}

// Chunk-major weights [c_out][chunks * 32] as a tiled map with a 32-column x `rows` box.
inline bool encode_w_tiled(const ConvParams& p, int rows, CUtensorMap* tm)
{
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(p.v2_chunks) * 32, static_cast<cuuint64_t>(p.c_out)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(p.v2_chunks) * 32 * 4};
    const cuuint32_t box[2] = {32, static_cast<cuuint32_t>(rows)};
    const cuuint32_t es[2] = {1, 1};
    return encoders().tiled(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(p.wt2), dims, strides, box, es,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Output [pixels][c_out] as a tiled map with a 32-channel x 32-pixel box (one warp's share).
inline bool encode_y_tiled(const ConvParams& p, CUtensorMap* tm)
{
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(p.c_out), static_cast<cuuint64_t>(p.pixels)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(p.c_out) * 4};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t es[2] = {1, 1};
    return encoders().tiled(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, p.y, dims, strides, box, es,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace nmtm
