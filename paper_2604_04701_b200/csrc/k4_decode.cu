// K4: decode path (M <= 16 tokens).  Same arithmetic as the tensor-core path (Eq. 7 + Eq. 3) but
// shaped for a memory-bound problem: W_q [N,K] is streamed once with 128-bit loads, one output
// channel n per warp at a time, the few token rows of Body_q are re-read from L1, products are
// accumulated with dp4a in int32 and the Aux correction c * sum_j Body_q[m,O_j] W_q[n,O_j] is
// added before the dequantizing store.
#include "kernels.h"

namespace muxq {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

template <int MT>
__global__ void __launch_bounds__(kThreads) k_decode(const DecodeArgs a) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int chunks = a.K >> 4;  // 16 codes per 128-bit load
    int r = 0;
    if (a.outlier_idx && a.n_outliers) r = min(__ldg(a.n_outliers), a.cap);
    const float sx0 = __ldg(a.s_x), sw0 = __ldg(a.s_w);

    for (int n = blockIdx.x * kWarps + warp; n < a.N; n += gridDim.x * kWarps) {
        const int8_t *wr = a.w_q + (size_t)n * a.ldw;
        int acc[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[m] = 0;
        for (int ch = lane; ch < chunks; ch += 32) {
            const uint4 w = __ldg(reinterpret_cast<const uint4 *>(wr) + ch);
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                if (m < a.M) {
                    const uint4 x = __ldg(reinterpret_cast<const uint4 *>(a.body_q + (size_t)m * a.ld_a) + ch);
                    acc[m] = __dp4a((int)x.x, (int)w.x, acc[m]);
                    acc[m] = __dp4a((int)x.y, (int)w.y, acc[m]);
                    acc[m] = __dp4a((int)x.z, (int)w.z, acc[m]);
                    acc[m] = __dp4a((int)x.w, (int)w.w, acc[m]);
                }
            }
        }
        // Aux term of Eq. 7 (shared scale: Aux_q == Body_q[:, O]), weighted by c = 2^exp - 1
        for (int j = lane; j < r; j += 32) {
            const int k = __ldg(a.outlier_idx + j);
            const int wv = wr[k];
#pragma unroll
            for (int m = 0; m < MT; ++m)
                if (m < a.M) acc[m] += a.c * wv * (int)a.body_q[(size_t)m * a.ld_a + k];
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc[m] += __shfl_xor_sync(0xffffffffu, acc[m], o);
        }
        const float sw = a.s_w_per_col ? __ldg(a.s_w + n) : sw0;
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            if (lane == m && m < a.M) {
                const float sx = a.s_x_per_row ? __ldg(a.s_x + m) : sx0;
                const size_t o = (size_t)m * a.ldy + n;
                if (a.out_kind == 2) {
                    reinterpret_cast<int32_t *>(a.Y)[o] = acc[m];
                } else {
                    float y = __fmul_rn(__fmul_rn(sx, sw), __int2float_rn(acc[m]));
                    if (a.bias) y = __fadd_rn(y, __ldg(a.bias + n));
                    if (a.out_kind == 1) reinterpret_cast<float *>(a.Y)[o] = y;
                    else reinterpret_cast<__half *>(a.Y)[o] = __float2half_rn(y);
                }
            }
        }
    }
}

}  // namespace

cudaError_t launch_decode(const DecodeArgs &a, cudaStream_t s) {
    int grid = (a.N + kWarps - 1) / kWarps;
    const int max_grid = num_sms() * 8;
    if (grid > max_grid) grid = max_grid;
    if (a.M <= 1) k_decode<1><<<grid, kThreads, 0, s>>>(a);
    else if (a.M <= 4) k_decode<4><<<grid, kThreads, 0, s>>>(a);
    else if (a.M <= 8) k_decode<8><<<grid, kThreads, 0, s>>>(a);
    else k_decode<16><<<grid, kThreads, 0, s>>>(a);
    return cudaGetLastError();
}

}  // namespace muxq
