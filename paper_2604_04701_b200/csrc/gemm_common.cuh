// Pieces shared by the INT8 GEMM kernels (one CTA per tile, and CTA pairs): tile constants, kernel
// parameters, the epilogue's convert-and-stage step, and the host-side tensor maps.
#pragma once
#include <cuda.h>

#include "kernels.h"
#include "ptx.cuh"

namespace muxq {
namespace gemm {

constexpr int BM = 128;
constexpr int BK = 128;  // bytes of K per stage = one 128-byte swizzle row
constexpr int kEpiWarps = 8;                       // two per TMEM lane quadrant, each half of the tile's columns
constexpr int kGemmThreads = 64 + 32 * kEpiWarps;  // TMA warp + MMA warp + epilogue warps
constexpr int kStatusTimeout = 6;  // MUXQ_ERR_TIMEOUT
constexpr int kOutF16 = 0, kOutF32 = 1, kOutI32 = 2;

struct GemmParams {
    int M, N, K;
    int tiles_m, tiles_n;
    int num_kb;    // body K blocks
    int has_aux;   // Aux operands present
    int c, cap;
    const int32_t *n_outliers;
    const float *s_x;
    const float *s_w;
    const float *bias;  // [N] fp32 or NULL: added to the dequantized value (one fp32 addition), then the cast
    int32_t *dev_status;
    int w_stable;  // the B operand may be read before the programmatic predecessor has finished
    uint32_t spin; // poll limit of the bounded waits
    int skip_kb;   // -1; a test names a K block whose loads are left out so that a wait runs out
};

// One 32-column chunk of one accumulator row: int32 -> fp32 (round to nearest even, exact below
// 2^24) -> times the scale [-> plus the layer's bias] -> output type, written as 16-byte pieces into the warp's staging row
// with the 128-byte swizzle the TMA store expects (16-byte piece g of row `lane` sits at g ^ (lane & 7)).
template <int kOut, bool kPerVec, bool kBias>
__device__ __forceinline__ void convert_chunk(const uint32_t (&v)[32], uint4 *srow, int piece0, uint32_t sw_xor,
                                              float sx, float sxw, const float *s_w_col, int cols_left,
                                              const float *bias_col) {
    if constexpr (kOut == kOutI32) {
#pragma unroll
        for (int g = 0; g < 8; ++g)
            srow[(piece0 + g) ^ sw_xor] = make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
    } else {
    float f[32];
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        float4 sc = make_float4(sxw, sxw, sxw, sxw);
        if (kPerVec) {
            // same address in every lane: one broadcast transaction; columns past N read as 0
            const float4 w = 4 * g < cols_left ? __ldg(reinterpret_cast<const float4 *>(s_w_col) + g)
                                               : make_float4(0.f, 0.f, 0.f, 0.f);
            sc = make_float4(__fmul_rn(sx, w.x), __fmul_rn(sx, w.y), __fmul_rn(sx, w.z), __fmul_rn(sx, w.w));
        }
        f[4 * g + 0] = __fmul_rn(sc.x, __int2float_rn((int)v[4 * g + 0]));
        f[4 * g + 1] = __fmul_rn(sc.y, __int2float_rn((int)v[4 * g + 1]));
        f[4 * g + 2] = __fmul_rn(sc.z, __int2float_rn((int)v[4 * g + 2]));
        f[4 * g + 3] = __fmul_rn(sc.w, __int2float_rn((int)v[4 * g + 3]));
        if constexpr (kBias) {  // same address in every lane: one broadcast transaction
            const float4 bb = 4 * g < cols_left ? __ldg(reinterpret_cast<const float4 *>(bias_col) + g)
                                                : make_float4(0.f, 0.f, 0.f, 0.f);
            f[4 * g + 0] = __fadd_rn(f[4 * g + 0], bb.x);
            f[4 * g + 1] = __fadd_rn(f[4 * g + 1], bb.y);
            f[4 * g + 2] = __fadd_rn(f[4 * g + 2], bb.z);
            f[4 * g + 3] = __fadd_rn(f[4 * g + 3], bb.w);
        }
    }
    if (kOut == kOutF32) {
#pragma unroll
        for (int g = 0; g < 8; ++g)
            srow[(piece0 + g) ^ sw_xor] = make_uint4(__float_as_uint(f[4 * g]), __float_as_uint(f[4 * g + 1]),
                                                     __float_as_uint(f[4 * g + 2]), __float_as_uint(f[4 * g + 3]));
    } else {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const __half2 h0 = __floats2half2_rn(f[8 * g + 0], f[8 * g + 1]);
            const __half2 h1 = __floats2half2_rn(f[8 * g + 2], f[8 * g + 3]);
            const __half2 h2 = __floats2half2_rn(f[8 * g + 4], f[8 * g + 5]);
            const __half2 h3 = __floats2half2_rn(f[8 * g + 6], f[8 * g + 7]);
            uint4 o;
            o.x = *reinterpret_cast<const uint32_t *>(&h0); o.y = *reinterpret_cast<const uint32_t *>(&h1);
            o.z = *reinterpret_cast<const uint32_t *>(&h2); o.w = *reinterpret_cast<const uint32_t *>(&h3);
            srow[(piece0 + g) ^ sw_xor] = o;
        }
    }
    }
}

// ---------------------------------------------------------------- host side: tensor maps + launch
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// int8 matrix [rows, cols] with pitch ld bytes, K-major; box = 128 bytes x box_rows, 128-byte swizzle.
// Out-of-range rows and columns read as zero, which a K tail or a ragged tile edge relies on.
inline bool make_map_i8(CUtensorMap *map, const void *ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld};
    cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// output matrix [M, N] of 2- or 4-byte elements, pitch ldy elements; box = 128 bytes x 32 rows
inline bool make_map_out(CUtensorMap *map, void *ptr, uint64_t rows, uint64_t cols, uint64_t ldy, int out_kind) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const uint64_t esz = out_kind == kOutF16 ? 2 : 4;
    const CUtensorMapDataType dt = out_kind == kOutF16   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                   : out_kind == kOutF32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                                         : CU_TENSOR_MAP_DATA_TYPE_INT32;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ldy * esz};
    cuuint32_t box[2] = {(cuuint32_t)(128 / esz), 32};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, dt, 2, ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace gemm
}  // namespace muxq
