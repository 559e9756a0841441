// K5: weight quantization (Eq. 2), per tensor or per output channel, storing W_q transposed as
// [N, K] with K contiguous -- the K-major B operand of the INT8 tensor-core GEMM.  Runs once per
// weight, off the per-layer hot path.
#include "kernels.h"

namespace muxq {

namespace {

constexpr int kTile = 32;

__global__ void __launch_bounds__(kTile * 8) k_quant_weight(const QuantWeightArgs a) {
    __shared__ int8_t tile[kTile][kTile + 4];
    const int tx = threadIdx.x, ty = threadIdx.y;  // 32 x 8
    const int n0 = blockIdx.x * kTile, k0 = blockIdx.y * kTile;
    const float qf = (float)a.qmax;
    const int n = n0 + tx;
    float s = 1.0f;
    if (n < a.N) {
        if (a.per_channel) {
            const float cm = __uint_as_float(a.colmax_bits[n]);
            s = cm > 0.0f ? __fdiv_rn(cm, qf) : 1.0f;
            if (blockIdx.y == 0 && ty == 0) a.s_w[n] = s;
        } else {
            s = *a.s_tensor;
            if (blockIdx.y == 0 && blockIdx.x == 0 && ty == 0 && tx == 0) a.s_w[0] = s;
        }
    }
#pragma unroll
    for (int i = 0; i < kTile; i += 8) {
        const int k = k0 + ty + i;
        int code = 0;
        if (k < a.K && n < a.N) {
            const float v = __half2float(a.W[(size_t)k * a.ldw + n]);
            float t = rintf(__fdiv_rn(v, s));
            t = fminf(fmaxf(t, -qf), qf);
            code = __float2int_rn(t);
        }
        tile[ty + i][tx] = (int8_t)code;  // [k][n]
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kTile; i += 8) {
        const int nn = n0 + ty + i, k = k0 + tx;
        if (nn < a.N && k < a.K) a.w_q[(size_t)nn * a.ld_q + k] = tile[tx][ty + i];
    }
}

}  // namespace

cudaError_t launch_quant_weight(const QuantWeightArgs &a, cudaStream_t s) {
    dim3 grid((a.N + kTile - 1) / kTile, (a.K + kTile - 1) / kTile), block(kTile, 8);
    k_quant_weight<<<grid, block, 0, s>>>(a);
    return cudaGetLastError();
}

}  // namespace muxq
