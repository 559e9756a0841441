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
// per-channel multipliers, Body abs-max -> s_X.
__device__ void detect_tail(const DetectArgs &a) {
    __shared__ int s_warp_cnt[kWarps];
    __shared__ float s_warp_max[kWarps];
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int K = a.K;
    int chunk = (K + kThreads - 1) / kThreads;
    chunk = (chunk + 7) & ~7;  // whole 8-channel groups per thread
    const int k0 = t * chunk;
    const int k1 = min(K, k0 + chunk);
    const float down = exp2f(-(float)a.exp_factor);

    int cnt = 0;
    for (int k = k0; k < k1; ++k) cnt += (__uint_as_float(__ldcg(a.colmax_bits + k)) > a.tau) ? 1 : 0;

    // exclusive prefix of cnt over the block (warp scan + warp totals)
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
    }
    if (lane == 31) s_warp_cnt[warp] = incl;
    __syncthreads();
    int base = 0, total = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        int c = s_warp_cnt[w];
        if (w < warp) base += c;
        total += c;
    }
    int pos = base + incl - cnt;

    float bmax = 0.0f;
    for (int g = k0; g < k1; g += 8) {
        uint8_t gf = 0;
        const int ge = min(k1, g + 8);
        for (int k = g; k < ge; ++k) {
            const float cm = __uint_as_float(__ldcg(a.colmax_bits + k));
            float mul = 1.0f;
            if (cm > a.tau) {
                if (pos < a.cap) {
                    a.outlier_idx[pos] = k;
                    mul = down;
                    gf = 1;
                }
                ++pos;
            }
            if (a.colmul) a.colmul[k] = mul;
            bmax = fmaxf(bmax, cm * mul);  // power-of-two scaling: exact
        }
        if (a.grpflag) a.grpflag[g >> 3] = gf;
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
        a.ctrl->n_outliers = total;
        if (a.n_outliers) *a.n_outliers = total;
        if (total > a.cap && a.dev_status) atomicMax(a.dev_status, kStatusCapacity);
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
        if (k < a.K && m > 0.0f) atomicMax(a.colmax_bits + k, __float_as_uint(m));
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

int num_sms() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
    }
    return n;
}

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
