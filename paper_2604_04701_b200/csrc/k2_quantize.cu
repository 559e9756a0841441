// K2: fused redistribute-and-quantize of the activations (Eq. 4-5 then Eq. 1), writing Body_q and
// the Aux block in the K-major INT8 layout the tensor-core GEMM consumes; the gather of W's outlier
// rows (needed by Aux.W in Eq. 7) rides in the same launch.  Also the real-domain decomposition
// used for inspection (muxq_build_aux).
//
// One warp per token row: 128-bit loads of 8 fp16, 64-bit stores of 8 codes.  Quantization uses a
// true fp32 division and round-half-to-even, so codes are reproducible bit for bit.
#include "kernels.h"

namespace muxq {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Eq. 1: code = clamp(round_half_even(v / s), -q, q)
__device__ __forceinline__ int quant1(float v, float s, float qf) {
    float t = rintf(__fdiv_rn(v, s));
    t = fminf(fmaxf(t, -qf), qf);
    return __float2int_rn(t);
}

__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8]) {
    const __half2 *h = reinterpret_cast<const __half2 *>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 p = __half22float2(h[i]);
        f[2 * i] = p.x;
        f[2 * i + 1] = p.y;
    }
}

template <bool PER_TOKEN>
__global__ void __launch_bounds__(kThreads) k_quant_act(const QuantActArgs a, int n_row_blocks) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float qf = (float)a.qmax;
    const int c = (1 << a.exp_factor) - 1;
    int r = 0;
    if (a.outlier_idx && a.n_outliers) r = min(__ldg(a.n_outliers), a.cap);

    if ((int)blockIdx.x >= n_row_blocks) {
        // ---- W_aux[n, c*j + t] = W_q[n, O_j]; zero beyond c*r.  4 bytes per thread.
        if (!a.w_aux) return;
        const int words_per_row = a.aux_cols >> 2;
        const int total = a.N * words_per_row;
        const int nthreads = (gridDim.x - n_row_blocks) * kThreads;
        for (int i = (blockIdx.x - n_row_blocks) * kThreads + threadIdx.x; i < total; i += nthreads) {
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
        return;
    }

    const int chunks = a.K >> 3;  // 8 channels per chunk
    const float down = exp2f(-(float)a.exp_factor);
    const float s_tensor = PER_TOKEN ? 1.0f : __ldg(a.s_x_tensor);
    for (int m = blockIdx.x * kWarps + warp; m < a.M; m += n_row_blocks * kWarps) {
        const __half *xr = a.X + (size_t)m * a.ldx;
        float s = s_tensor;
        if (PER_TOKEN) {
            // per-token scale from Body's row (after the 2^-e redistribution)
            float mx = 0.0f;
            for (int ch = lane; ch < chunks; ch += 32) {
                const uint4 v = __ldg(reinterpret_cast<const uint4 *>(xr) + ch);
                float f[8];
                unpack8(v, f);
                if (a.grpflag && a.grpflag[ch]) {
                    const float4 m0 = __ldg(reinterpret_cast<const float4 *>(a.colmul) + 2 * ch);
                    const float4 m1 = __ldg(reinterpret_cast<const float4 *>(a.colmul) + 2 * ch + 1);
                    f[0] *= m0.x; f[1] *= m0.y; f[2] *= m0.z; f[3] *= m0.w;
                    f[4] *= m1.x; f[5] *= m1.y; f[6] *= m1.z; f[7] *= m1.w;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) mx = fmaxf(mx, fabsf(f[i]));
            }
            mx = warp_max(mx);
            s = mx > 0.0f ? __fdiv_rn(mx, qf) : 1.0f;
            if (lane == 0) a.s_x_rows[m] = s;
        }
        for (int ch = lane; ch < chunks; ch += 32) {
            const uint4 v = __ldg(reinterpret_cast<const uint4 *>(xr) + ch);
            float f[8];
            unpack8(v, f);
            if (a.grpflag && a.grpflag[ch]) {
                const float4 m0 = __ldg(reinterpret_cast<const float4 *>(a.colmul) + 2 * ch);
                const float4 m1 = __ldg(reinterpret_cast<const float4 *>(a.colmul) + 2 * ch + 1);
                f[0] *= m0.x; f[1] *= m0.y; f[2] *= m0.z; f[3] *= m0.w;
                f[4] *= m1.x; f[5] *= m1.y; f[6] *= m1.z; f[7] *= m1.w;
            }
            uint32_t lo = 0, hi = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                lo |= (uint32_t)(quant1(f[i], s, qf) & 0xff) << (8 * i);
                hi |= (uint32_t)(quant1(f[4 + i], s, qf) & 0xff) << (8 * i);
            }
            *reinterpret_cast<uint2 *>(a.body_q + (size_t)m * a.ld_q + ch * 8) = make_uint2(lo, hi);
        }
        if (a.aux_q) {
            // Aux block: column c*j + t holds the code of Body[m, O_j] (Eq. 5), shared scale.
            for (int w = lane; w < (a.aux_cols >> 2); w += 32) {
                uint32_t packed = 0;
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const int j = (w * 4 + b) / c;
                    if (j < r) {
                        const float v = __half2float(xr[__ldg(a.outlier_idx + j)]) * down;
                        packed |= (uint32_t)(quant1(v, s, qf) & 0xff) << (8 * b);
                    }
                }
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
    int n_row_blocks = (a.M + kWarps - 1) / kWarps;
    const int max_blocks = num_sms() * 8;
    if (n_row_blocks > max_blocks) n_row_blocks = max_blocks;
    int gather_blocks = 0;
    if (a.w_aux) {
        gather_blocks = (a.N * (a.aux_cols >> 2) + kThreads - 1) / kThreads;
        if (gather_blocks > 64) gather_blocks = 64;
    }
    const int grid = n_row_blocks + gather_blocks;
    if (a.per_token)
        k_quant_act<true><<<grid, kThreads, 0, s>>>(a, n_row_blocks);
    else
        k_quant_act<false><<<grid, kThreads, 0, s>>>(a, n_row_blocks);
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
