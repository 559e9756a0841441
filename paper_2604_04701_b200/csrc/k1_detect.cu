// K1: per-channel abs-max of X, outlier-channel detection (Section III-C criterion), ascending
// compaction of the outlier set O, Body abs-max and the per-tensor scale of Eq. 1.
//
// Memory-bound: X is read once with 128-bit loads (a warp covers 256 consecutive channels of one
// token row).  Maxima of non-negative floats are order-independent, so partial maxima are merged
// with integer atomicMax on the bit patterns; the last CTA to finish runs the tail.
#include "kernels.h"

namespace muxq {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kColsPerBlock = 256;  // 32 lanes x 8 fp16 (one 16-byte load each)
constexpr int kStatusCapacity = 5;  // MUXQ_ERR_CAPACITY

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Tail, run by one CTA once every partial maximum is merged: threshold, ordered compaction,
// per-channel multipliers, Body abs-max -> s_X.  Rounds of 2048 channels: thread t owns the 8
// consecutive channels [base + 8t, base + 8t + 8), loaded with two coalesced 128-bit loads.
__device__ void detect_tail(const DetectArgs &a) {
    __shared__ int s_warp_cnt[kWarps];
    __shared__ float s_warp_max[kWarps];
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int K = a.K;
    const float down = exp2f(-(float)a.exp_factor);
    int carry = 0;
    float bmax = 0.0f;
    for (int base = 0; base < K; base += kThreads * 8) {
        const int k0 = base + t * 8;
        const bool active = k0 < K;  // K % 8 == 0: a group is entirely inside or outside
        float cm[8];
        if (active) {
            const float4 v0 = __ldcg(reinterpret_cast<const float4 *>(a.colmax_bits + k0));
            const float4 v1 = __ldcg(reinterpret_cast<const float4 *>(a.colmax_bits + k0) + 1);
            cm[0] = v0.x; cm[1] = v0.y; cm[2] = v0.z; cm[3] = v0.w;
            cm[4] = v1.x; cm[5] = v1.y; cm[6] = v1.z; cm[7] = v1.w;
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) cm[i] = 0.0f;
        }
        int cnt = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) cnt += (cm[i] > a.tau) ? 1 : 0;
        // exclusive prefix of cnt over the block (warp scan + warp totals)
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += n;
        }
        if (lane == 31) s_warp_cnt[warp] = incl;
        __syncthreads();
        int before = 0, total = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const int c = s_warp_cnt[w];
            if (w < warp) before += c;
            total += c;
        }
        int pos = carry + before + incl - cnt;
        if (active) {
            float mul[8];
            uint8_t gf = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                mul[i] = 1.0f;
                if (cm[i] > a.tau) {
                    if (pos < a.cap) {
                        a.outlier_idx[pos] = k0 + i;
                        mul[i] = down;
                        gf = 1;
                    }
                    ++pos;
                }
                bmax = fmaxf(bmax, cm[i] * mul[i]);  // power-of-two scaling: exact
            }
            if (a.colmul) {
                reinterpret_cast<float4 *>(a.colmul + k0)[0] = make_float4(mul[0], mul[1], mul[2], mul[3]);
                reinterpret_cast<float4 *>(a.colmul + k0)[1] = make_float4(mul[4], mul[5], mul[6], mul[7]);
            }
            if (a.grpflag) a.grpflag[k0 >> 3] = gf;
        }
        carry += total;
        __syncthreads();  // s_warp_cnt is reused by the next round
    }
    bmax = warp_max(bmax);
    if (lane == 0) s_warp_max[warp] = bmax;
    __syncthreads();
    if (t == 0) {
        float m = 0.0f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) m = fmaxf(m, s_warp_max[w]);
        const float s = m > 0.0f ? __fdiv_rn(m, (float)a.qmax) : 1.0f;  // Eq. 1
        if (a.s_x) *a.s_x = s;
        a.ctrl->s_x = s;
        a.ctrl->inv_s_x = __fdiv_rn(1.0f, s);
        a.ctrl->n_outliers = carry;
        if (a.n_outliers) *a.n_outliers = carry;
        if (carry > a.cap && a.dev_status) atomicMax(a.dev_status, kStatusCapacity);
    }
}

__global__ void __launch_bounds__(kThreads) k_colabsmax_detect(const DetectArgs a, int rows_per_block) {
    __shared__ float s_part[kWarps][kColsPerBlock];
    __shared__ int s_is_last;
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int col = blockIdx.x * kColsPerBlock + lane * 8;
    const int row_begin = blockIdx.y * rows_per_block;
    const int row_end = min(a.M, row_begin + rows_per_block);

    __half2 m0 = __float2half2_rn(0.f), m1 = m0, m2 = m0, m3 = m0;
    if (col < a.K) {
        const __half *p = a.X + (size_t)col;
        int r = row_begin + warp;
        for (; r + 3 * kWarps < row_end; r += 4 * kWarps) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                v[u] = __ldg(reinterpret_cast<const uint4 *>(p + (size_t)(r + u * kWarps) * a.ldx));
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                m0 = __hmax2(m0, __habs2(*reinterpret_cast<__half2 *>(&v[u].x)));
                m1 = __hmax2(m1, __habs2(*reinterpret_cast<__half2 *>(&v[u].y)));
                m2 = __hmax2(m2, __habs2(*reinterpret_cast<__half2 *>(&v[u].z)));
                m3 = __hmax2(m3, __habs2(*reinterpret_cast<__half2 *>(&v[u].w)));
            }
        }
        for (; r < row_end; r += kWarps) {
            uint4 v = __ldg(reinterpret_cast<const uint4 *>(p + (size_t)r * a.ldx));
            m0 = __hmax2(m0, __habs2(*reinterpret_cast<__half2 *>(&v.x)));
            m1 = __hmax2(m1, __habs2(*reinterpret_cast<__half2 *>(&v.y)));
            m2 = __hmax2(m2, __habs2(*reinterpret_cast<__half2 *>(&v.z)));
            m3 = __hmax2(m3, __habs2(*reinterpret_cast<__half2 *>(&v.w)));
        }
    }
    float *sp = &s_part[warp][lane * 8];
    sp[0] = __low2float(m0); sp[1] = __high2float(m0);
    sp[2] = __low2float(m1); sp[3] = __high2float(m1);
    sp[4] = __low2float(m2); sp[5] = __high2float(m2);
    sp[6] = __low2float(m3); sp[7] = __high2float(m3);
    __syncthreads();
    {
        float m = 0.0f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) m = fmaxf(m, s_part[w][t]);
        const int k = blockIdx.x * kColsPerBlock + t;
        // most CTAs find the running maximum already at or above theirs and skip the atomic
        if (k < a.K && m > 0.0f && __float_as_uint(m) > __ldcg(a.colmax_bits + k))
            atomicMax(a.colmax_bits + k, __float_as_uint(m));
    }
    // last CTA to arrive runs the tail
    __threadfence();
    __syncthreads();
    if (t == 0) {
        const unsigned total = gridDim.x * gridDim.y;
        s_is_last = (atomicAdd(&a.ctrl->blocks_done, 1u) == total - 1u);
    }
    __syncthreads();
    if (s_is_last) {
        __threadfence();
        detect_tail(a);
    }
}

__global__ void __launch_bounds__(kThreads) k_detect_tail_only(const DetectArgs a) { detect_tail(a); }

}  // namespace

cudaError_t launch_detect(const DetectArgs &a, cudaStream_t s) {
    const int col_blocks = (a.K + kColsPerBlock - 1) / kColsPerBlock;
    int slices = (num_sms() * 6 + col_blocks - 1) / col_blocks;
    int rows_per_block = (a.M + slices - 1) / slices;
    if (rows_per_block < 4 * kWarps) rows_per_block = 4 * kWarps;
    slices = (a.M + rows_per_block - 1) / rows_per_block;
    dim3 grid(col_blocks, slices);
    k_colabsmax_detect<<<grid, kThreads, 0, s>>>(a, rows_per_block);
    return cudaGetLastError();
}

cudaError_t launch_detect_finalize(const DetectArgs &a, cudaStream_t s) {
    k_detect_tail_only<<<1, kThreads, 0, s>>>(a);
    return cudaGetLastError();
}

}  // namespace muxq
