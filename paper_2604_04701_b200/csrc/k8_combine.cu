// Own-scale reading of Eq. 7: Body and Aux are quantized with different scales, so their INT8 products cannot share
// an integer accumulator.  The two products are dequantized separately (Eq. 3: t1 = (s_X s_W) acc_b,
// t2 = (s_A s_W) acc_a, both by the GEMM kernel's fp32 epilogue) and joined here: Y = t1 + c * t2, in that order of
// operations, then cast.  A plain streaming kernel; this reading is provided for completeness, not tuned.
#include "kernels.h"

namespace muxq {

namespace {

__global__ void __launch_bounds__(256) k_combine(const CombineArgs a) {
    const size_t n4 = ((size_t)a.M * a.N) >> 2;  // N % 8 == 0: rows are whole float4s
    const float cf = (float)a.c;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        const float4 u = reinterpret_cast<const float4 *>(a.t1)[i];
        const float4 v = reinterpret_cast<const float4 *>(a.t2)[i];
        float4 y;
        y.x = __fadd_rn(u.x, __fmul_rn(cf, v.x));
        y.y = __fadd_rn(u.y, __fmul_rn(cf, v.y));
        y.z = __fadd_rn(u.z, __fmul_rn(cf, v.z));
        y.w = __fadd_rn(u.w, __fmul_rn(cf, v.w));
        const size_t e = i << 2, row = e / a.N, col = e - row * a.N;
        if (a.out_f16) {
            __half2 *o = reinterpret_cast<__half2 *>(reinterpret_cast<__half *>(a.Y) + row * a.ldy + col);
            o[0] = __floats2half2_rn(y.x, y.y);
            o[1] = __floats2half2_rn(y.z, y.w);
        } else {
            *reinterpret_cast<float4 *>(reinterpret_cast<float *>(a.Y) + row * a.ldy + col) = y;
        }
    }
}

}  // namespace

cudaError_t launch_combine(const CombineArgs &a, cudaStream_t s) {
    const size_t n4 = ((size_t)a.M * a.N) >> 2;
    int grid = (int)((n4 + 255) / 256);
    const int cap = num_sms() * 8;
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    k_combine<<<grid, 256, 0, s>>>(a);
    return cudaGetLastError();
}

}  // namespace muxq
