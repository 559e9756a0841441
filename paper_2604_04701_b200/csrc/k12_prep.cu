// Fused activation preparation for muxq_linear: per-channel abs-max and outlier detection
// (Section III-C), the redistribution of Eq. 4-5 and the abs-max quantization of Eq. 1, in ONE
// launch that reads X from HBM once.
//
// The per-tensor scale and the outlier set depend on every row of X, so the kernel has two passes
// separated by a grid-wide barrier.  It is launched cooperatively with one CTA per SM; CTA b owns a
// contiguous slab of token rows and keeps it in shared memory between the passes (a slab of
// M/148 rows x K fp16 fits for the GPT-2 shapes; rows that do not fit are re-read, normally from L2):
//   pass 1  stream the slab (128-bit loads, a thread owns 8 channels and walks down the rows),
//           stash it in shared memory, merge channel maxima CTA-wide in shared memory and then
//           device-wide with integer atomicMax on the bit patterns (maxima of non-negative floats
//           are order independent, so the result is exact).  The device-wide accumulators are
//           replicated kColmaxReplicas times (CTA b uses copy b mod R): same-address atomics
//           serialise in L2, and one copy would take 148 of them per channel
//   barrier bounded spin on an arrival counter; a time-out raises MUXQ_ERR_TIMEOUT, marks the workspace (the
//           counter keeps its top bit until muxq_workspace_init clears it, and every later call that finds
//           the mark fails at once instead of computing on half-merged maxima) and returns
//   pass 2  every CTA derives the channel factors and s_X from the K maxima (cheap, redundant; warp 0
//           lists O meanwhile), then quantizes its slab out of shared memory with the pass-1 thread
//           mapping (per tensor) or one warp per token row (per token), writing Body_q, the Aux block
//           and (spread over the grid) the gathered W_aux rows.
// The kernel expects the barrier counter, the reader counter and the replicated accumulators to be zero and
// leaves them zero: once every CTA has fetched the merged maxima (each takes a ticket after doing so; the
// holder of the last ticket knows), nothing reads them any more, and that CTA clears them during the last phase.
// A call therefore needs no separate clearing step; a barrier time-out leaves them dirty (and marked).
#include <mutex>

#include "kernels.h"
#include "quant.cuh"

namespace muxq {

namespace {

constexpr int kT = 1024;  // the warp-group split of the last phase (512 + 256 + 256 threads) assumes this
constexpr int kWarps = kT / 32;
constexpr int kMaxK = 8 * kT;  // one group of 8 channels per thread
static_assert(kMaxK == kPrepMaxK, "the accumulator region of the workspace is sized for kPrepMaxK channels");
constexpr int kColmaxReplicas = kPrepColmaxReplicas;
constexpr int kStatusCapacity = 5;  // MUXQ_ERR_CAPACITY
constexpr int kStatusTimeout = 6;   // MUXQ_ERR_TIMEOUT
constexpr uint32_t kBarrierSpin = 1u << 21;
constexpr uint32_t kPoisonBit = 0x80000000u;  // in Ctrl::arrived: an earlier call on this workspace timed out
constexpr int kMaxDynSmem = 227 * 1024 - 1024;

__host__ __device__ inline int fixed_smem_bytes(int K, int cap, int aux_cols) {
    const int G = K >> 3;
    // colmul | colmax | group flags | outlier indices [cap] | source channel of every Aux column [aux_cols]
    return 8 * K + ((G + 15) & ~15) + ((cap + 3) & ~3) * 4 + ((aux_cols * 2 + 15) & ~15);
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void absmax4(__half2 (&m)[4], const uint4 &v) {
    m[0] = __hmax2(m[0], __habs2(*reinterpret_cast<const __half2 *>(&v.x)));
    m[1] = __hmax2(m[1], __habs2(*reinterpret_cast<const __half2 *>(&v.y)));
    m[2] = __hmax2(m[2], __habs2(*reinterpret_cast<const __half2 *>(&v.z)));
    m[3] = __hmax2(m[3], __habs2(*reinterpret_cast<const __half2 *>(&v.w)));
}

// 8 values of one 16-byte chunk, channel factors applied when the group holds an outlier channel
__device__ __forceinline__ void load_chunk(const uint4 *src, int ch, const uint8_t *flag, const float *colmul,
                                           float (&f)[8]) {
    const uint4 v = src[ch];
    unpack8(v, f);
    if (flag[ch]) {
        const float4 m0 = reinterpret_cast<const float4 *>(colmul)[2 * ch];
        const float4 m1 = reinterpret_cast<const float4 *>(colmul)[2 * ch + 1];
        f[0] *= m0.x; f[1] *= m0.y; f[2] *= m0.z; f[3] *= m0.w;  // 1 or 2^-e: exact
        f[4] *= m1.x; f[5] *= m1.y; f[6] *= m1.z; f[7] *= m1.w;
    }
}

// kAllFit: the host has sized the slab for every row of the largest CTA share, so the loops over rows that
// live only in global memory are compiled out (and with them their registers).
// kPerToken: per-token scales (one warp per row in pass 2) instead of the per-tensor scale; one instantiation
// per granularity keeps the other one's code out of the kernel.
template <bool kAllFit, bool kPerToken>
__global__ void __launch_bounds__(kT, 1) k_prep(const PrepArgs a, int rows_base, int rows_extra, int slab_bytes,
                                                int rstride, uint32_t g_magic, uint32_t spin, uint32_t extra_arrivals) {
    extern __shared__ __align__(16) uint8_t smem[];
    __shared__ float s_warp_max[kWarps];
    __shared__ int s_r_true;
    __shared__ int s_fail;
    __shared__ int s_last;
    __shared__ float s_aux_scale;  // per-tensor Aux scale (own-scale reading)

    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int K = a.K, G = K >> 3;
    float *s_colmul = reinterpret_cast<float *>(smem);
    uint32_t *s_colmax = reinterpret_cast<uint32_t *>(smem + 4 * K);
    uint8_t *s_flag = smem + 8 * K;
    int32_t *s_oidx = reinterpret_cast<int32_t *>(smem + 8 * K + ((G + 15) & ~15));
    uint16_t *s_auxsrc = reinterpret_cast<uint16_t *>(s_oidx + ((a.cap + 3) & ~3));
    uint8_t *slab = smem + fixed_smem_bytes(K, a.cap, a.aux_cols);

    const int b = blockIdx.x;
    const int r0 = b * rows_base + min(b, rows_extra);
    const int rows = rows_base + (b < rows_extra ? 1 : 0);
    const int fit = kAllFit ? rows : min(rows, slab_bytes / (2 * K));

    // ---------------------------------------------------------------- pass 1: channel maxima
    // CTA-wide maxima of pass 1 accumulate in s_part, laid out [channel within group][group] so that the lanes of a
    // warp (consecutive groups) hit consecutive banks; with the natural [group][channel] layout every shared-memory
    // atomic of a warp would be an 8-way bank conflict.  It shares its bytes with s_colmul, which is written only
    // after the grid barrier.
    uint32_t *s_part = reinterpret_cast<uint32_t *>(smem);
    for (int k = t; k < K; k += kT) s_part[k] = 0u;
    __syncthreads();
    {
        // thread = (row offset, channel group); rstride = kT / G row offsets are in use (G <= kT).  The division
        // t / G is a multiplication by g_magic = ceil(2^20 / G), exact for t < 1024 (t * G < 2^20); both constants
        // come from the host: with 32 warps per SM every instruction of per-thread set-up costs 8 cycles of SM time,
        // and a 32-bit division is some 25 instructions
        const int row_off = (int)(((uint32_t)t * g_magic) >> 20), cg = t - row_off * G;
        if (row_off < rstride) {
            __half2 m[4];
            m[0] = m[1] = m[2] = m[3] = __float2half2_rn(0.f);
            // up to 8 independent 16-byte loads in flight per thread; addresses advance by constant steps
            const size_t xstep = (size_t)rstride * a.ldx;
            const uint32_t sstep = (uint32_t)rstride * (uint32_t)K * 2u;
            const __half *px = a.X + ((size_t)r0 + row_off) * a.ldx + cg * 8;
            uint8_t *ps = slab + (size_t)row_off * K * 2 + cg * 16;
            for (int row = row_off; row < rows; row += 8 * rstride) {
                uint4 v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u)
                    v[u] = row + u * rstride < rows ? __ldg(reinterpret_cast<const uint4 *>(px + u * xstep))
                                                    : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    absmax4(m, v[u]);
                    if (row + u * rstride < fit) *reinterpret_cast<uint4 *>(ps + u * sstep) = v[u];
                }
                px += 8 * xstep;
                ps += 8 * sstep;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float lo = __low2float(m[i]), hi = __high2float(m[i]);
                atomicMax(&s_part[(2 * i) * G + cg], __float_as_uint(lo));  // non-negative: bit patterns order like values
                atomicMax(&s_part[(2 * i + 1) * G + cg], __float_as_uint(hi));
            }
        }
    }
    __syncthreads();
    {
        uint32_t *rep = a.colmax_rep + (size_t)(b % kColmaxReplicas) * K;
        for (int k = t; k < K; k += kT) {
            // a warp's 32 consecutive channels travel as one 128-byte reduction request
            const uint32_t v = s_part[(k & 7) * G + (k >> 3)];
            if (v != 0u) atomicMax(rep + k, v);
        }
    }

    // ---------------------------------------------------------------- grid-wide barrier (bounded)
    __syncthreads();
    if (t == 0) {
        __threadfence();  // cumulative: publishes the whole CTA's reductions, ordered before it by the barrier
        atomicAdd(&a.ctrl->arrived, 1u);
        bool ok = false;
        const uint32_t want = gridDim.x + extra_arrivals;  // (extra arrivals: a test's way of making this wait run out)
        // acquire loads: once the full count is seen, the other CTAs' reductions (released before their
        // arrivals) are visible to this thread, and through the barrier below to the whole CTA.  A set top bit
        // means an earlier call on this workspace timed out and left the counters dirty.
        for (uint32_t i = 0; i < spin; ++i) {
            const uint32_t v = ld_acquire_u32(&a.ctrl->arrived);
            if (v & kPoisonBit) break;
            if (v >= want) { ok = true; break; }
        }
        s_fail = ok ? 0 : 1;
        if (!ok) {
            atomicOr(&a.ctrl->arrived, kPoisonBit);
            if (a.dev_status) atomicMax(a.dev_status, kStatusTimeout);
        }
    }
    __syncthreads();
    if (s_fail) return;

    // ---------------------------------------------------------------- channel factors and s_X (every CTA)
    const float down = __int_as_float((127 - a.exp_factor) << 23);  // 2^-e
    const float qf = (float)a.qmax;
    const int c = (1 << a.exp_factor) - 1;
    // Aux layout: with the shared scale every Aux column is repeated c times (one accumulator serves Eq. 7); with its
    // own scale Aux is a separate product and its columns are stored once
    const int crep = a.aux_own ? 1 : c;
    // channel maxima = max over the replicas, fetched with coalesced 16-byte loads
    for (int k4 = t; k4 < (K >> 2); k4 += kT) {
        uint4 v[kColmaxReplicas];
#pragma unroll
        for (int rp = 0; rp < kColmaxReplicas; ++rp)
            v[rp] = __ldcg(reinterpret_cast<const uint4 *>(a.colmax_rep + (size_t)rp * K) + k4);
        uint4 mx = v[0];
#pragma unroll
        for (int rp = 1; rp < kColmaxReplicas; ++rp) {
            mx.x = max(mx.x, v[rp].x); mx.y = max(mx.y, v[rp].y);
            mx.z = max(mx.z, v[rp].z); mx.w = max(mx.w, v[rp].w);
        }
        reinterpret_cast<uint4 *>(s_colmax)[k4] = mx;
        if (b == 0) reinterpret_cast<uint4 *>(a.colmax_bits)[k4] = mx;
    }
    __syncthreads();
    // This CTA holds its copy of the maxima.  The CTA that takes the last ticket knows that every CTA does
    // (and has therefore left the barrier), so it may put the accumulators and both counters back to zero for
    // the next call; the ticket is taken by the last warp, which is off the critical path of the quantization.
    // (No fence: the loads above have returned their values, so stores issued after the last ticket was
    // taken cannot reach them.)
    // Every thread derives the factors of the 8 channels it owns in both passes: 2^-e where the channel
    // holds an element above the threshold (strict), else 1.  (When more channels are flagged than the
    // capacity allows the call fails with MUXQ_ERR_CAPACITY and Y is unspecified, so no ordering is needed here.)
    const int row_off = (int)(((uint32_t)t * g_magic) >> 20), cg = t - row_off * G;
    float mul[8];
    uint32_t fmask = 0;  // bit i: channel 8*cg + i is an outlier channel
    {
        const float4 v0 = reinterpret_cast<const float4 *>(s_colmax)[2 * cg];
        const float4 v1 = reinterpret_cast<const float4 *>(s_colmax)[2 * cg + 1];
        const float cm[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
        float bmax = 0.0f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const bool flagged = cm[i] > a.tau;
            mul[i] = flagged ? down : 1.0f;
            fmask |= flagged ? (1u << i) : 0u;
            bmax = fmaxf(bmax, cm[i] * mul[i]);  // power-of-two scaling: exact
        }
        if (row_off == 0) {  // shared copies: the outlier listing below and the per-token path read them
            reinterpret_cast<float4 *>(s_colmul)[2 * cg] = make_float4(mul[0], mul[1], mul[2], mul[3]);
            reinterpret_cast<float4 *>(s_colmul)[2 * cg + 1] = make_float4(mul[4], mul[5], mul[6], mul[7]);
            s_flag[cg] = (uint8_t)fmask;
        }
        bmax = warp_max(bmax);
        if (lane == 0) s_warp_max[warp] = bmax;
    }
    __syncthreads();
    float s, inv_s;
    {
        const float mx = warp_max(s_warp_max[lane]);
        s = mx > 0.0f ? __fdiv_rn(mx, qf) : 1.0f;  // Eq. 1
        inv_s = __frcp_rn(s);  // correctly rounded 1/s
        if (b == 0 && t == 0) {
            a.ctrl->s_x = s;
            a.ctrl->inv_s_x = inv_s;
        }
    }
    // The last warp (idle or lightly loaded in the quantization loop) lists O in ascending order from the
    // per-group flag masks; nothing needs the list before the Aux block.  It also fills the source channel
    // of every Aux column: column c*j + i mirrors channel O_j (Eq. 5), repeated c times for Eq. 7.
    if (warp == kWarps - 1) {
        uint32_t ticket = 0;
        if (lane == 0) ticket = atomicAdd(&a.ctrl->readers, 1u);  // every thread passed the barrier after the fetch
        int carry = 0;
        for (int base = 0; base < G; base += 32) {
            const int g = base + lane;
            uint32_t m = g < G ? s_flag[g] : 0u;
            if (!__any_sync(0xffffffffu, m != 0u)) continue;
            const int cnt = __popc(m);
            int incl = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int n = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += n;
            }
            int pos = carry + incl - cnt;
            while (m) {
                const int i = __ffs(m) - 1;
                m &= m - 1;
                if (pos < a.cap) {
                    s_oidx[pos] = 8 * g + i;
                    if (b == 0) a.outlier_idx[pos] = 8 * g + i;
                }
                ++pos;
            }
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        __syncwarp();
        // (a.aux_cols == 0: no Aux block and no W_aux wanted, the list of sources has no room and no reader)
        const int ucols = min(crep * min(carry, a.cap), a.aux_cols);
        for (int i = lane; i < ucols; i += 32) s_auxsrc[i] = (uint16_t)s_oidx[i / crep];
        // own-scale reading, per tensor: max |Aux| = 2^-e times the largest maximum among the listed channels
        float am = 0.0f;
        for (int j = lane; j < min(carry, a.cap); j += 32) am = fmaxf(am, __uint_as_float(s_colmax[s_oidx[j]]) * down);
        am = warp_max(am);
        if (lane == 0) {
            s_last = ticket == gridDim.x - 1 ? 1 : 0;
            s_r_true = carry;
            s_aux_scale = am > 0.0f ? __fdiv_rn(am, qf) : 1.0f;
            if (b == 0) {
                a.ctrl->s_a = s_aux_scale;
                a.ctrl->n_outliers = carry;
                if (carry > a.cap && a.dev_status) atomicMax(a.dev_status, kStatusCapacity);
            }
        }
    }
    if (kPerToken) __syncthreads();  // the per-token path reads the shared factor copies and the Aux sources

    // Let a kernel launched as a programmatic dependent (the GEMM) start its set-up on SMs as they free up;
    // it still waits for this whole grid to finish before it reads anything written here.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---------------------------------------------------------------- pass 2: Body_q and the Aux block
    if (!kPerToken) {
        // Per-tensor scale: the pass-1 mapping again (a thread owns 8 channels and walks down the
        // rows), so the channel factors stay in registers and consecutive lanes store consecutive codes.
        if (row_off < rstride) {
            // brackets of 1/s with the channel factor folded in (power of two: exact)
            float blo[8], bhi[8];
            {
                float lo, hi;
                recip_bracket(inv_s, lo, hi);
#pragma unroll
                for (int i = 0; i < 8; ++i) { blo[i] = lo * mul[i]; bhi[i] = hi * mul[i]; }
            }
            // 8 values of this thread's channel group -> 8 codes; the exact division only next to a tie
            auto codes = [&](const uint4 &v) -> uint2 {
                float f[8];
                unpack8(v, f);
                uint32_t code[8];
                if (quant8_bracket(f, blo, bhi, code)) return codes_exact(v, fmask, down, s, qf);  // next to a tie: rare
                return pack8(code);
            };
            // Rows row_off, row_off + rstride, ...: first those held in the slab, two per iteration, then the
            // rest from global memory (normally L2), four loads in flight.  Addresses advance by constant steps.
            const uint32_t sstep = (uint32_t)rstride * (uint32_t)K * 2u;
            const size_t qstep = (size_t)rstride * a.ld_q, xstep = (size_t)rstride * a.ldx;
            const uint8_t *sp = slab + (size_t)row_off * K * 2 + cg * 16;
            int8_t *qp = a.body_q + ((size_t)r0 + row_off) * a.ld_q + cg * 8;
            int row = row_off;
            for (; row + rstride < fit; row += 2 * rstride) {
                const uint4 v0 = *reinterpret_cast<const uint4 *>(sp);
                const uint4 v1 = *reinterpret_cast<const uint4 *>(sp + sstep);
                *reinterpret_cast<uint2 *>(qp) = codes(v0);
                *reinterpret_cast<uint2 *>(qp + qstep) = codes(v1);
                sp += 2 * sstep;
                qp += 2 * qstep;
            }
            if (row < fit) {
                *reinterpret_cast<uint2 *>(qp) = codes(*reinterpret_cast<const uint4 *>(sp));
                qp += qstep;
                row += rstride;
            }
            // The rows that did not fit the slab come from global memory again, LAST row first: pass 1 read them in
            // ascending order, so the highest rows are the ones most likely still in L2 when X is larger than L2
            // (the slab holds the lowest rows, the first to be evicted).  Four loads in flight; addresses step down
            // by constant amounts.
            if (!kAllFit && row < rows) {
                const int cnt = (rows - row + rstride - 1) / rstride;  // rows of this thread outside the slab
                const __half *xp = a.X + ((size_t)r0 + row) * a.ldx + cg * 8 + (size_t)(cnt - 1) * xstep;
                qp += (size_t)(cnt - 1) * qstep;
                for (int k = cnt - 1; k >= 0; k -= 4) {
                    uint4 v[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        v[u] = k - u >= 0 ? __ldg(reinterpret_cast<const uint4 *>(xp - u * xstep))
                                          : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        if (k - u >= 0) *reinterpret_cast<uint2 *>(qp - u * qstep) = codes(v[u]);
                    }
                    xp -= 4 * xstep;
                    qp -= 4 * qstep;
                }
            }
        }
    } else {
        const int r = min(s_r_true, a.cap);
        const int used_cols = crep * r, pad_words = a.aux_own ? a.aux_cols >> 2 : ((used_cols + 31) & ~31) >> 2;
        // A row is walked by a whole warp, or by half a warp when the CTA has more rows than warps: two rounds of
        // rows per warp would run every reduction, division and store latency of a row twice in sequence.
        const int lpr = rows > kWarps ? 16 : 32;  // lanes per row
        const int rpw = 32 / lpr, sub = lane / lpr, l = lane - sub * lpr;
        auto part_max = [&](float v) {  // over the lanes of one row
            for (int o = lpr >> 1; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
            return v;
        };
        for (int base = warp * rpw; base < rows; base += kWarps * rpw) {  // warp-uniform trip count
            const int row = min(base + sub, rows - 1);
            const bool live = base + sub < rows;  // the other half of the warp may have run out of rows
            const size_t m = (size_t)r0 + row;
            const uint4 *src = row < fit ? reinterpret_cast<const uint4 *>(slab + (size_t)row * K * 2)
                                         : reinterpret_cast<const uint4 *>(a.X + m * a.ldx);
            // per-token scale from Body's row (after the 2^-e redistribution)
            float mx = 0.0f;
            for (int ch = l; ch < G; ch += lpr) {
                float f[8];
                load_chunk(src, ch, s_flag, s_colmul, f);
#pragma unroll
                for (int i = 0; i < 8; ++i) mx = fmaxf(mx, fabsf(f[i]));
            }
            mx = part_max(mx);
            const float sr = mx > 0.0f ? __fdiv_rn(mx, qf) : 1.0f;
            float rlo, rhi;
            recip_bracket(__frcp_rn(sr), rlo, rhi);
            if (l == 0 && live) a.s_x_rows[m] = sr;
            int8_t *q = a.body_q + m * a.ld_q;
            for (int ch = l; ch < G && live; ch += lpr) {
                float f[8];
                load_chunk(src, ch, s_flag, s_colmul, f);
                uint32_t code[8];
                if (quant8_bracket(f, rlo, rhi, code)) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) code[i] = (uint32_t)quant_exact(f[i], sr, qf);
                }
                *reinterpret_cast<uint2 *>(q + ch * 8) = pack8(code);
            }
            if (a.aux_q && !a.aux_own) {
                // shared scale: Aux_q[m, c*j + i] is the code Body_q[m, O_j] these lanes have just written
                __syncwarp();
                for (int w = l; w < pad_words && live; w += lpr) {
                    uint32_t packed = 0;
#pragma unroll
                    for (int bb = 0; bb < 4; ++bb)
                        if (w * 4 + bb < used_cols)
                            packed |= (uint32_t)(uint8_t)q[s_auxsrc[w * 4 + bb]] << (8 * bb);
                    *reinterpret_cast<uint32_t *>(a.aux_q + m * a.ld_aux + w * 4) = packed;
                }
            } else if (a.aux_q) {
                // own scale per token: s_A[m] = max_j |Aux[m, j]| / q, then Eq. 1 on Aux[m, j] = X[m, O_j] * 2^-e
                const __half *xr = reinterpret_cast<const __half *>(src);
                float am = 0.0f;
                for (int j = l; j < used_cols; j += lpr) am = fmaxf(am, fabsf(__half2float(xr[s_auxsrc[j]]) * down));
                am = part_max(am);
                const float sa = am > 0.0f ? __fdiv_rn(am, qf) : 1.0f;
                if (l == 0 && live) a.s_a_rows[m] = sa;
                for (int w = l; w < pad_words && live; w += lpr) {
                    uint32_t packed = 0;
#pragma unroll
                    for (int bb = 0; bb < 4; ++bb)
                        if (w * 4 + bb < used_cols)
                            packed |= (uint32_t)(quant_exact(__half2float(xr[s_auxsrc[w * 4 + bb]]) * down, sa, qf) & 0xff)
                                      << (8 * bb);
                    *reinterpret_cast<uint32_t *>(a.aux_q + m * a.ld_aux + w * 4) = packed;
                }
            }
        }
    }

    // ---------------------------------------------------------------- Aux block (per tensor) and W_aux
    __syncthreads();  // the last warp's outlier list and Aux sources are complete
    const int r = min(s_r_true, a.cap);
    const int used_cols = crep * r;
    // The GEMM consumes the Aux columns in steps of 32, i.e. columns [0, pad_cols); an Aux column of zeros makes the
    // matching W_aux column irrelevant and vice versa, so both blocks are written up to pad_cols only (codes, then
    // zeros) and the columns behind are left as they are.
    // (With its own scale Aux is the A operand of a product over all aux_cols columns: zeros to the end.)
    const int pad_words = a.aux_own ? a.aux_cols >> 2 : ((used_cols + 31) & ~31) >> 2;
    const float s_codes = a.aux_own ? s_aux_scale : s;
    // i / pad_words below as a multiplication where the item counts are small (i < 2^22: the float holds i + 0.5
    // exactly, and (i + 0.5) / pad_words is at least 0.5 / pad_words away from an integer, far more than the rounding
    // of the product); a 32-bit division is some 25 instructions, and this phase is one or two items per thread
    const float inv_pad = 1.0f / (float)max(pad_words, 1);
    const bool small_counts = (long long)max(rows, a.N) * pad_words < (1ll << 22);
    auto div_pad = [&](int i) { return small_counts ? (int)(((float)i + 0.5f) * inv_pad) : i / max(pad_words, 1); };
    // Independent jobs share the CTA's warps so that their latencies overlap instead of adding up: warps 0-15 the
    // Aux codes, warps 16-31 the W_aux gather (and, in one CTA per launch, the clean-up for the next call).
    const bool do_aux = a.aux_q && !kPerToken;
    // Aux codes by the bracket test too (2^-e folded into the brackets), the exact division only next to a tie
    float alo, ahi;
    recip_bracket(__frcp_rn(s_codes), alo, ahi);
    alo *= down;
    ahi *= down;
    if (warp < 16) {
        if (do_aux) {
            // Aux_q[m, c*j + i] = code of Body[m, O_j] (Eq. 5, shared scale), recomputed from the slab with the
            // exact division, one 4-byte word per thread and round
            for (int i = t; i < rows * pad_words; i += 512) {
                const int row = div_pad(i), w = i - row * pad_words;
                const size_t m = (size_t)r0 + row;
                const __half *xr = row < fit ? reinterpret_cast<const __half *>(slab + (size_t)row * K * 2)
                                             : a.X + m * a.ldx;
                uint32_t packed = 0;
#pragma unroll
                for (int bb = 0; bb < 4; ++bb) {
                    const int col = w * 4 + bb;
                    if (col < used_cols) {
                        const float xv = __half2float(xr[s_auxsrc[col]]);
                        const uint32_t ca = __float_as_uint(fmaf(xv, ahi, 12582912.0f));
                        const uint32_t cb = __float_as_uint(fmaf(xv, alo, 12582912.0f));
                        const uint32_t code = ca == cb ? ca : (uint32_t)quant_exact(xv * down, s_codes, qf);
                        packed |= (code & 0xffu) << (8 * bb);
                    }
                }
                *reinterpret_cast<uint32_t *>(a.aux_q + m * a.ld_aux + w * 4) = packed;
            }
        }
    } else {
        if (s_last && warp < 24) {
            uint4 *rep4 = reinterpret_cast<uint4 *>(a.colmax_rep);
            for (int i = t - 512; i < kColmaxReplicas * (K >> 2); i += 256) rep4[i] = make_uint4(0u, 0u, 0u, 0u);
            if (t == 512) {
                a.ctrl->arrived = 0u;
                a.ctrl->readers = 0u;
            }
        }
        if (a.w_aux) {
            // W_aux[n, c*j + i] = W_q[n, O_j], one 4-byte word per thread and round, spread over the grid
            const int total = a.N * pad_words;
            for (int i = b * 512 + (t - 512); i < total; i += gridDim.x * 512) {
                const int n = div_pad(i), w = i - n * pad_words;
                uint32_t packed = 0;
#pragma unroll
                for (int bb = 0; bb < 4; ++bb)
                    if (w * 4 + bb < used_cols)
                        packed |= (uint32_t)(uint8_t)a.w_q[(size_t)n * a.ldw + s_auxsrc[w * 4 + bb]] << (8 * bb);
                *reinterpret_cast<uint32_t *>(a.w_aux + (size_t)n * a.ld_waux + w * 4) = packed;
            }
        }
    }
}

}  // namespace

bool prep_supported(int M, int K) { return M >= 1 && K >= 8 && K % 8 == 0 && K <= kMaxK; }

cudaError_t launch_prep(const PrepArgs &a, cudaStream_t s) {
    static const void *const fns[4] = {
        reinterpret_cast<const void *>(k_prep<false, false>), reinterpret_cast<const void *>(k_prep<false, true>),
        reinterpret_cast<const void *>(k_prep<true, false>), reinterpret_cast<const void *>(k_prep<true, true>)};
    static PerDevice<int> attr_set;
    const int dev = current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    {
        std::lock_guard<std::mutex> lock(device_mutex());
        if (!attr_set.have[dev]) {
            for (const void *f : fns) {
                cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
                if (e != cudaSuccess) return e;
            }
            attr_set.have[dev] = true;
        }
    }
    int grid = num_sms();
    if (grid < 1) return cudaErrorInvalidDevice;
    if (grid > a.M) grid = a.M;
    int rows_base = a.M / grid, rows_extra = a.M % grid;
    const int rows_max = rows_base + (rows_extra ? 1 : 0);
    const int fixed = fixed_smem_bytes(a.K, a.cap, a.aux_cols);
    const long long want = (long long)rows_max * a.K * 2;
    int slab_bytes = (int)(want < (long long)(kMaxDynSmem - fixed) ? want : (long long)(kMaxDynSmem - fixed));
    slab_bytes &= ~15;
    PrepArgs args = a;
    const int G = a.K >> 3;
    int rstride = kT / G;
    uint32_t g_magic = ((1u << 20) + (uint32_t)G - 1u) / (uint32_t)G;
    uint32_t spin = test_hooks().spin_limit ? test_hooks().spin_limit : kBarrierSpin;
    uint32_t extra_arrivals = test_hooks().prep_extra_arrivals;
    void *params[] = {&args, &rows_base, &rows_extra, &slab_bytes, &rstride, &g_magic, &spin, &extra_arrivals};
    const bool all_fit = (long long)slab_bytes >= want;
    const void *fn = fns[(all_fit ? 2 : 0) + (a.per_token ? 1 : 0)];
    return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kT), params, (size_t)(fixed + slab_bytes), s);
}

}  // namespace muxq
