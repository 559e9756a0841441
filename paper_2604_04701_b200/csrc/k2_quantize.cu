// K2: fused redistribute-and-quantize of the activations (Eq. 4-5 then Eq. 1), writing Body_q and
// the Aux block in the K-major INT8 layout the tensor-core GEMM consumes; the gather of W's outlier
// rows (needed by Aux.W in Eq. 7) rides in the same launch.  Also the real-domain decomposition
// used for inspection (muxq_build_aux).
//
// 128-bit loads of 8 fp16, 64-bit stores of 8 codes.  Codes equal round_half_even(v / s) with a
// true fp32 division bit for bit; a reciprocal multiply pre-screens the (common) values that are
// provably far from a rounding tie, the rest take the division.
#include "kernels.h"
#include "quant.cuh"

namespace muxq {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

// Aux block word w of row xr: columns 4w..4w+3, column c*j + t holds the code of Body[m, O_j]
__device__ __forceinline__ uint32_t aux_word(const __half *xr, const int32_t *oidx, int w, int c, int r, float down,
                                             float s, float qf) {
    uint32_t packed = 0;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        const int j = (w * 4 + b) / c;
        if (j < r) {
            const float v = __half2float(xr[__ldg(oidx + j)]) * down;
            packed |= (uint32_t)(quant_exact(v, s, qf) & 0xff) << (8 * b);
        }
    }
    return packed;
}

// W_aux[n, c*j + t] = W_q[n, O_j]; zero beyond c*r.  4 bytes per thread.
__device__ __forceinline__ void gather_w_aux(const QuantActArgs &a, int r, int c, int tid, int nthreads) {
    const int words_per_row = a.aux_cols >> 2;
    const int total = a.N * words_per_row;
    for (int i = tid; i < total; i += nthreads) {
        const int n = i / words_per_row, w = i - n * words_per_row;
        uint32_t packed = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int j = (w * 4 + b) / c;
            if (j < r) {
                const int8_t v = a.w_q[(size_t)n * a.ldw + __ldg(a.outlier_idx + j)];
                packed |= (uint32_t)(uint8_t)v << (8 * b);
            }
        }
        *reinterpret_cast<uint32_t *>(a.w_aux + (size_t)n * a.ld_waux + w * 4) = packed;
    }
}

// Per-tensor scale.  Grid: [main blocks | Aux blocks | W_aux blocks].  Main blocks follow the K1
// layout (a warp spans 256 consecutive channels, the CTA's warps walk down the rows), so each
// thread keeps its 8 channel factors in registers for all its rows.
__global__ void __launch_bounds__(kThreads)
k_quant_act_tensor(const QuantActArgs a, int col_blocks, int row_slices, int rows_per_block, int aux_blocks) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float qf = (float)a.qmax;
    const int c = (1 << a.exp_factor) - 1;
    int r = 0;
    if (a.outlier_idx && a.n_outliers) r = min(__ldg(a.n_outliers), a.cap);
    const float s = __ldg(a.s_x_tensor);
    const int main_blocks = col_blocks * row_slices;
    const int b = blockIdx.x;

    if (b < main_blocks) {
        const float inv_s = __ldg(a.inv_s_x_tensor);
        const int cb = b % col_blocks, slice = b / col_blocks;
        const int col = cb * 256 + lane * 8;
        if (col >= a.K) return;
        float mul[8];
        if (a.colmul) {
            const float4 m0 = __ldg(reinterpret_cast<const float4 *>(a.colmul + col));
            const float4 m1 = __ldg(reinterpret_cast<const float4 *>(a.colmul + col) + 1);
            mul[0] = m0.x; mul[1] = m0.y; mul[2] = m0.z; mul[3] = m0.w;
            mul[4] = m1.x; mul[5] = m1.y; mul[6] = m1.z; mul[7] = m1.w;
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) mul[i] = 1.0f;
        }
        const int row_begin = slice * rows_per_block;
        const int row_end = min(a.M, row_begin + rows_per_block);
        const __half *p = a.X + col;
        int8_t *q = a.body_q + col;
        int m = row_begin + warp;
        for (; m + 3 * kWarps < row_end; m += 4 * kWarps) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                v[u] = __ldg(reinterpret_cast<const uint4 *>(p + (size_t)(m + u * kWarps) * a.ldx));
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float f[8];
                unpack8(v[u], f);
#pragma unroll
                for (int i = 0; i < 8; ++i) f[i] *= mul[i];  // 1 or 2^-e: exact
                *reinterpret_cast<uint2 *>(q + (size_t)(m + u * kWarps) * a.ld_q) = quant8(f, s, inv_s, qf);
            }
        }
        for (; m < row_end; m += kWarps) {
            const uint4 v = __ldg(reinterpret_cast<const uint4 *>(p + (size_t)m * a.ldx));
            float f[8];
            unpack8(v, f);
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] *= mul[i];
            *reinterpret_cast<uint2 *>(q + (size_t)m * a.ld_q) = quant8(f, s, inv_s, qf);
        }
        return;
    }
    if (b < main_blocks + aux_blocks) {
        // ---- Aux block rows (Eq. 5), one 4-byte word per thread
        const int words = a.aux_cols >> 2;
        const int total = a.M * words;
        const float down = exp2f(-(float)a.exp_factor);
        const int used_words = (c * r + 3) >> 2;
        for (int i = (b - main_blocks) * kThreads + threadIdx.x; i < total; i += aux_blocks * kThreads) {
            const int m = i / words, w = i - m * words;
            uint32_t packed = 0;
            if (w < used_words) packed = aux_word(a.X + (size_t)m * a.ldx, a.outlier_idx, w, c, r, down, s, qf);
            *reinterpret_cast<uint32_t *>(a.aux_q + (size_t)m * a.ld_aux + w * 4) = packed;
        }
        return;
    }
    if (a.w_aux)
        gather_w_aux(a, r, c, (b - main_blocks - aux_blocks) * kThreads + threadIdx.x,
                     (gridDim.x - main_blocks - aux_blocks) * kThreads);
}

// Per-token scales: one warp per token row (row abs-max by warp shuffle, then the codes).
__global__ void __launch_bounds__(kThreads) k_quant_act_token(const QuantActArgs a, int n_row_blocks) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float qf = (float)a.qmax;
    const int c = (1 << a.exp_factor) - 1;
    int r = 0;
    if (a.outlier_idx && a.n_outliers) r = min(__ldg(a.n_outliers), a.cap);

    if ((int)blockIdx.x >= n_row_blocks) {
        if (a.w_aux)
            gather_w_aux(a, r, c, (blockIdx.x - n_row_blocks) * kThreads + threadIdx.x,
                         (gridDim.x - n_row_blocks) * kThreads);
        return;
    }
    const int chunks = a.K >> 3;  // 8 channels per chunk
    const float down = exp2f(-(float)a.exp_factor);
    for (int m = blockIdx.x * kWarps + warp; m < a.M; m += n_row_blocks * kWarps) {
        const __half *xr = a.X + (size_t)m * a.ldx;
        // per-token scale from Body's row (after the 2^-e redistribution)
        float mx = 0.0f;
        for (int ch0 = 0; ch0 < chunks; ch0 += 128) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int ch = ch0 + u * 32 + lane;
                v[u] = ch < chunks ? __ldg(reinterpret_cast<const uint4 *>(xr) + ch) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int ch = ch0 + u * 32 + lane;
                float f[8];
                unpack8(v[u], f);
                if (ch < chunks && a.grpflag && a.grpflag[ch]) {
                    const float4 m0 = __ldg(reinterpret_cast<const float4 *>(a.colmul) + 2 * ch);
                    const float4 m1 = __ldg(reinterpret_cast<const float4 *>(a.colmul) + 2 * ch + 1);
                    f[0] *= m0.x; f[1] *= m0.y; f[2] *= m0.z; f[3] *= m0.w;
                    f[4] *= m1.x; f[5] *= m1.y; f[6] *= m1.z; f[7] *= m1.w;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) mx = fmaxf(mx, fabsf(f[i]));
            }
        }
        mx = warp_max(mx);
        const float s = mx > 0.0f ? __fdiv_rn(mx, qf) : 1.0f;
        const float inv_s = __fdiv_rn(1.0f, s);
        if (lane == 0) a.s_x_rows[m] = s;
        for (int ch0 = 0; ch0 < chunks; ch0 += 128) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int ch = ch0 + u * 32 + lane;
                v[u] = ch < chunks ? __ldg(reinterpret_cast<const uint4 *>(xr) + ch) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int ch = ch0 + u * 32 + lane;
                if (ch >= chunks) continue;
                float f[8];
                unpack8(v[u], f);
                if (a.grpflag && a.grpflag[ch]) {
                    const float4 m0 = __ldg(reinterpret_cast<const float4 *>(a.colmul) + 2 * ch);
                    const float4 m1 = __ldg(reinterpret_cast<const float4 *>(a.colmul) + 2 * ch + 1);
                    f[0] *= m0.x; f[1] *= m0.y; f[2] *= m0.z; f[3] *= m0.w;
                    f[4] *= m1.x; f[5] *= m1.y; f[6] *= m1.z; f[7] *= m1.w;
                }
                *reinterpret_cast<uint2 *>(a.body_q + (size_t)m * a.ld_q + ch * 8) = quant8(f, s, inv_s, qf);
            }
        }
        if (a.aux_q) {
            const int used_words = (c * r + 3) >> 2;
            for (int w = lane; w < (a.aux_cols >> 2); w += 32) {
                uint32_t packed = 0;
                if (w < used_words) packed = aux_word(xr, a.outlier_idx, w, c, r, down, s, qf);
                *reinterpret_cast<uint32_t *>(a.aux_q + (size_t)m * a.ld_aux + w * 4) = packed;
            }
        }
    }
}

// Real-domain Body / Aux (Eq. 4, Eq. 5) in fp32.
__global__ void __launch_bounds__(kThreads) k_build_aux(const BuildAuxArgs a) {
    const int r = min(__ldg(a.n_outliers), a.cap);
    const float down = exp2f(-(float)a.exp_factor);
    const size_t stride = (size_t)gridDim.x * kThreads;
    const size_t tid = (size_t)blockIdx.x * kThreads + threadIdx.x;
    for (size_t i = tid; i < (size_t)a.M * a.cap; i += stride) {
        const int m = (int)(i / a.cap), j = (int)(i - (size_t)m * a.cap);
        a.aux[(size_t)m * a.ld_aux + j] =
            j < r ? __half2float(a.X[(size_t)m * a.ldx + a.outlier_idx[j]]) * down : 0.0f;
    }
    if (a.body) {
        for (size_t i = tid; i < (size_t)a.M * a.K; i += stride) {
            const int m = (int)(i / a.K), k = (int)(i - (size_t)m * a.K);
            a.body[(size_t)m * a.ld_body + k] = __half2float(a.X[(size_t)m * a.ldx + k]);
        }
    }
}
// second pass (after the copy above is complete in stream order): scale the outlier columns
__global__ void __launch_bounds__(kThreads) k_build_aux_scale_body(const BuildAuxArgs a) {
    const int r = min(__ldg(a.n_outliers), a.cap);
    const float down = exp2f(-(float)a.exp_factor);
    const size_t stride = (size_t)gridDim.x * kThreads;
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < (size_t)a.M * r; i += stride) {
        const int m = (int)(i / r), j = (int)(i - (size_t)m * r);
        const int k = a.outlier_idx[j];
        a.body[(size_t)m * a.ld_body + k] = __half2float(a.X[(size_t)m * a.ldx + k]) * down;
    }
}

}  // namespace

cudaError_t launch_quant_act(const QuantActArgs &a, cudaStream_t s) {
    int gather_blocks = 0;
    if (a.w_aux) {
        gather_blocks = (a.N * (a.aux_cols >> 2) + kThreads - 1) / kThreads;
        if (gather_blocks > 64) gather_blocks = 64;
    }
    if (a.per_token) {
        int n_row_blocks = (a.M + kWarps - 1) / kWarps;
        const int max_blocks = num_sms() * 8;
        if (n_row_blocks > max_blocks) n_row_blocks = max_blocks;
        k_quant_act_token<<<n_row_blocks + gather_blocks, kThreads, 0, s>>>(a, n_row_blocks);
        return cudaGetLastError();
    }
    const int col_blocks = (a.K + 255) / 256;
    int slices = (num_sms() * 6 + col_blocks - 1) / col_blocks;
    int rows_per_block = (a.M + slices - 1) / slices;
    if (rows_per_block < 4 * kWarps) rows_per_block = 4 * kWarps;
    slices = (a.M + rows_per_block - 1) / rows_per_block;
    int aux_blocks = 0;
    if (a.aux_q) {
        aux_blocks = (a.M * (a.aux_cols >> 2) + kThreads - 1) / kThreads;
        if (aux_blocks > num_sms() * 2) aux_blocks = num_sms() * 2;
    }
    k_quant_act_tensor<<<col_blocks * slices + aux_blocks + gather_blocks, kThreads, 0, s>>>(a, col_blocks, slices,
                                                                                           rows_per_block, aux_blocks);
    return cudaGetLastError();
}

cudaError_t launch_build_aux(const BuildAuxArgs &a, cudaStream_t s) {
    size_t work = (size_t)a.M * (a.body ? a.K : a.cap);
    int grid = (int)((work + kThreads - 1) / kThreads);
    if (grid > num_sms() * 16) grid = num_sms() * 16;
    if (grid < 1) grid = 1;
    k_build_aux<<<grid, kThreads, 0, s>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || !a.body) return e;
    k_build_aux_scale_body<<<grid, kThreads, 0, s>>>(a);
    return cudaGetLastError();
}

}  // namespace muxq
