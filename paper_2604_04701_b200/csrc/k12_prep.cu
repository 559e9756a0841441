// Fused activation preparation for muxq_linear: per-channel abs-max and outlier detection
// (Section III-C), the redistribution of Eq. 4-5 and the abs-max quantization of Eq. 1, in ONE
// launch.
//
// The per-tensor scale and the outlier set depend on every row of X, so the kernel has two passes
// separated by a grid-wide barrier.  It is launched cooperatively with one CTA per SM; CTA b owns a
// contiguous slab of token rows.  Both passes are built around one ring of row stripes in shared
// memory that a producer warp fills with bulk asynchronous copies (one per token row, completion on an
// mbarrier per stripe) while the other 31 warps consume:
//   stripe   nrow = floor(992 / (K/8)) consecutive rows; consumer thread (row_off, cg) owns the 16-byte
//            chunk of channels 8cg..8cg+7 of row row_off of every stripe, so its channel maxima (pass 1)
//            and its channel factors (pass 2) stay in registers
//   pass 1   stripes 0..T-1 stream through the ring (S slots); a thread folds its chunk into its 8
//            running maxima.  The ring ends up holding the LAST S stripes.  Channel maxima are merged
//            CTA-wide in shared memory and device-wide with integer atomicMax on the bit patterns
//            (maxima of non-negative floats are order independent, so the result is exact), into
//            accumulators replicated kColmaxReplicas times (CTA b uses copy b mod R: same-address
//            atomics serialise in L2)
//   barrier  bounded spin on an arrival counter; a time-out raises MUXQ_ERR_TIMEOUT, marks the workspace
//            (the counter keeps its top bit until muxq_workspace_init clears it) and returns
//   pass 2   every CTA derives the channel factors and s_X from the K maxima (cheap, redundant; the
//            producer warp lists O meanwhile), then quantizes: first the stripes still resident, in
//            place, then the evicted ones, which the producer fetches again in REVERSE order -- the most
//            recently evicted stripe is the one most likely still in L2 -- into slots as they are
//            freed.  A thread writes the 8 codes of its chunk to Body_q, and, where its chunk holds an
//            outlier channel, the copies of those codes that make up the Aux block (Eq. 5).  Per-token
//            scales take one warp per token row instead (rows not resident are read from global memory).
//            The producer warp gathers this CTA's share of W_aux before it starts fetching.
// The kernel expects the barrier counter, the reader counter and the replicated accumulators to be zero
// and leaves them zero: once every CTA has fetched the merged maxima (each takes a ticket after doing so;
// the holder of the last ticket knows), nothing reads them any more, and that CTA clears them at its end.
// A call therefore needs no separate clearing step.
#include <mutex>

#include "kernels.h"
#include "ptx.cuh"
#include "quant.cuh"

namespace muxq {

namespace {

constexpr int kT = 1024;
constexpr int kWarps = kT / 32;
constexpr int kConsWarps = kWarps - 1;      // warp kWarps-1 is the producer
constexpr int kConsThreads = 32 * kConsWarps;
constexpr int kMaxG = kConsThreads;         // one group of 8 channels per consumer thread
constexpr int kMaxSlots = 32;
constexpr int kColmaxReplicas = kPrepColmaxReplicas;
constexpr int kStatusCapacity = 5;  // MUXQ_ERR_CAPACITY
constexpr int kStatusTimeout = 6;   // MUXQ_ERR_TIMEOUT
constexpr uint32_t kPoisonBit = 0x80000000u;  // in Ctrl::arrived: an earlier call on this workspace timed out
constexpr int kMaxDynSmem = 227 * 1024 - 2048;

__host__ __device__ inline int fixed_smem_bytes(int K, int cap, int aux_cols) {
    const int G = K >> 3;
    // colmul | colmax | group flags | rank of each group's first outlier channel [G] u16 | outlier indices [cap] |
    // source channel of every Aux column [aux_cols] u16; rounded so that the ring behind it is 128-byte aligned
    const int n = 8 * K + ((G + 15) & ~15) + ((2 * G + 15) & ~15) + ((cap + 3) & ~3) * 4 + ((aux_cols * 2 + 15) & ~15);
    return (n + 127) & ~127;
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// One token row (or any 16-byte-aligned span) global -> shared, completion counted in bytes on an mbarrier.
__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gsrc, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// Bounded wait of a whole converged warp with a caller-chosen limit (the default limit is far above any
// legitimate wait; a test shortens it to make a wait run out).
__device__ __forceinline__ bool wait_warp(uint64_t *bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i) {
        if (__any_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
        if ((i & 63u) == 63u && __any_sync(0xffffffffu, *abort_flag != 0u)) return false;
    }
    *abort_flag = 1u;
    return false;
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

// Geometry of one launch, computed on the host.
struct PrepGeom {
    int rows_base, rows_extra;  // CTA b owns rows_base (+1 if b < rows_extra) rows
    int nrow;                   // rows per stripe
    int slots;                  // S: stripes the ring holds
    uint32_t g_magic;           // ceil(2^20 / G): t / G as a multiplication, exact for t < 1024
    uint32_t spin;              // poll limit of every bounded wait
    uint32_t extra_arrivals;    // 0; a test sets it to make the grid barrier wait for arrivals that never come
};

// kPerToken: per-token scales (one warp per row in pass 2) instead of the per-tensor scale; one instantiation
// per granularity keeps the other one's code out of the kernel.
template <bool kPerToken>
__global__ void __launch_bounds__(kT, 1) k_prep(const PrepArgs a, const PrepGeom g) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ uint64_t bar_full[kMaxSlots], bar_empty[kMaxSlots];
    __shared__ float s_warp_max[kWarps];
    __shared__ int s_r_true;
    __shared__ uint32_t s_abort;
    __shared__ int s_last;
    __shared__ volatile int s_list_ready;
    __shared__ float s_aux_scale;  // per-tensor Aux scale (own-scale reading)

    const int t = threadIdx.x, lane = t & 31;
    const int warp = __shfl_sync(0xffffffffu, t >> 5, 0);  // warp-uniform by construction
    const int K = a.K, G = K >> 3;
    float *s_colmul = reinterpret_cast<float *>(smem);
    uint32_t *s_colmax = reinterpret_cast<uint32_t *>(smem + 4 * K);
    uint8_t *s_flag = smem + 8 * K;
    uint16_t *s_rank = reinterpret_cast<uint16_t *>(smem + 8 * K + ((G + 15) & ~15));
    int32_t *s_oidx = reinterpret_cast<int32_t *>(reinterpret_cast<uint8_t *>(s_rank) + ((2 * G + 15) & ~15));
    uint16_t *s_auxsrc = reinterpret_cast<uint16_t *>(s_oidx + ((a.cap + 3) & ~3));
    uint8_t *ring = smem + fixed_smem_bytes(K, a.cap, a.aux_cols);

    const int b = blockIdx.x;
    const int r0 = b * g.rows_base + min(b, g.rows_extra);
    const int rows = g.rows_base + (b < g.rows_extra ? 1 : 0);
    const int nrow = g.nrow, S = g.slots;
    const int T = (rows + nrow - 1) / nrow;          // stripes of this CTA
    const int Sres = min(S, T);                      // stripes resident after pass 1
    const uint32_t row_bytes = (uint32_t)K * 2u;
    const uint32_t slot_bytes = (uint32_t)nrow * row_bytes;
    volatile uint32_t *abort_flag = &s_abort;
    const bool producer = warp == kWarps - 1;

    // consumer thread = (row offset inside a stripe, channel group)
    const int row_off = (int)(((uint32_t)t * g.g_magic) >> 20), cg = t - row_off * G;
    const bool active = !producer && row_off < nrow;

    // CTA-wide maxima of pass 1 accumulate in s_part, laid out [channel within group][group] so that the lanes of a
    // warp (consecutive groups) hit consecutive banks.  It shares its bytes with s_colmul, written after the barrier.
    uint32_t *s_part = reinterpret_cast<uint32_t *>(smem);
    for (int k = t; k < K; k += kT) s_part[k] = 0u;
    if (t == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&bar_full[s], 1);            // the producer's expect_tx arrival; bytes from the copies
            mbar_init(&bar_empty[s], kConsWarps);  // one arrival per consumer warp
        }
        s_abort = 0u;
        s_list_ready = 0;
        fence_barrier_init();
    }
    __syncthreads();

    // Fetch of stripe `stripe` (rows stripe*nrow ...) into ring position n % S, load number n of this CTA.
    auto issue = [&](int n, int stripe) -> bool {
        const int slot = n % S;
        if (n >= S && !wait_warp(&bar_empty[slot], (uint32_t)((n / S) - 1) & 1u, abort_flag, g.spin)) return false;
        const int first = stripe * nrow, cnt = min(nrow, rows - first);
        if (lane == 0) mbar_expect_tx(&bar_full[slot], (uint32_t)cnt * row_bytes);
        __syncwarp();
        for (int i = lane; i < cnt; i += 32)
            bulk_load(ring + (size_t)slot * slot_bytes + (size_t)i * row_bytes,
                      a.X + ((size_t)r0 + first + i) * a.ldx, row_bytes, &bar_full[slot]);
        return true;
    };
    // After a time-out the copies already issued must land before this CTA's shared memory is released.
    auto drain = [&](int issued) {
        for (int n = max(0, issued - S); n < issued; ++n) {
            const int slot = n % S;
            for (uint32_t i = 0; i < g.spin; ++i)
                if (__any_sync(0xffffffffu, mbar_try_wait(&bar_full[slot], (uint32_t)(n / S) & 1u))) break;
        }
    };

    // ---------------------------------------------------------------- pass 1: channel maxima
    int issued = 0;  // producer warp: loads issued so far (drained after a time-out)
    if (producer) {
        for (; issued < T; ++issued)
            if (!issue(issued, issued)) break;
    } else {
        __half2 m[4];
        m[0] = m[1] = m[2] = m[3] = __float2half2_rn(0.f);
        const uint8_t *mine = ring + (size_t)row_off * row_bytes + cg * 16;
        bool ok = true;
        for (int n = 0; n < T && ok; ++n) {
            const int slot = n % S;
            ok = wait_warp(&bar_full[slot], (uint32_t)(n / S) & 1u, abort_flag, g.spin);
            if (!ok) break;
            if (active && n * nrow + row_off < rows)
                absmax4(m, *reinterpret_cast<const uint4 *>(mine + (size_t)slot * slot_bytes));
            if (n + S < T) {  // this position is fetched into again during pass 1
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar_empty[slot]);
            }
        }
        if (active) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float lo = __low2float(m[i]), hi = __high2float(m[i]);
                atomicMax(&s_part[(2 * i) * G + cg], __float_as_uint(lo));  // non-negative: bit patterns order like values
                atomicMax(&s_part[(2 * i + 1) * G + cg], __float_as_uint(hi));
            }
        }
    }
    __syncthreads();
    if (s_abort) {  // a wait of pass 1 ran out: let the copies in flight land, mark the workspace, leave
        if (producer) drain(issued);
        __syncthreads();
        if (t == 0) {
            atomicOr(&a.ctrl->arrived, kPoisonBit);
            if (a.dev_status) atomicMax(a.dev_status, kStatusTimeout);
        }
        return;
    }
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
        const uint32_t want = gridDim.x + g.extra_arrivals;
        // acquire loads: once the full count is seen, the other CTAs' reductions (released before their
        // arrivals) are visible to this thread, and through the barrier below to the whole CTA.  A set top
        // bit means an earlier call on this workspace timed out and left the counters dirty.
        for (uint32_t i = 0; i < g.spin; ++i) {
            const uint32_t v = ld_acquire_u32(&a.ctrl->arrived);
            if (v & kPoisonBit) break;
            if (v >= want) { ok = true; break; }
        }
        if (!ok) {
            s_abort = 1u;
            atomicOr(&a.ctrl->arrived, kPoisonBit);
            if (a.dev_status) atomicMax(a.dev_status, kStatusTimeout);
        }
    }
    __syncthreads();
    if (s_abort) return;

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
    // the next call.  (No fence: the loads above have returned their values, so stores issued after the last
    // ticket was taken cannot reach them.)
    // Every thread derives the factors of the 8 channels it owns in both passes: 2^-e where the channel
    // holds an element above the threshold (strict), else 1.
    float mul[8];
    uint32_t fmask = 0;  // bit i: channel 8*cg + i is an outlier channel
    {
        // (every thread has a valid channel group; the copies held by threads beyond the stripe mapping are unused)
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
        if (row_off == 0) {  // shared copies: the outlier listing and the per-token path read them
            // (s_part, which shares its bytes with s_colmul, was last read before the grid barrier)
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

    // Let a kernel launched as a programmatic dependent (the GEMM) start its set-up on SMs as they free up;
    // it still waits for this whole grid to finish before it reads anything written here.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (producer) {
        // -------------------------------------------------------------- outlier list, Aux sources, W_aux, refetches
        uint32_t ticket = 0;
        if (lane == 0) ticket = atomicAdd(&a.ctrl->readers, 1u);  // every thread passed the barrier after the fetch
        int carry = 0;
        for (int base = 0; base < G; base += 32) {
            const int gi = base + lane;
            uint32_t mk = gi < G ? s_flag[gi] : 0u;
            if (!__any_sync(0xffffffffu, mk != 0u)) continue;
            const int cnt = __popc(mk);
            int incl = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int nn = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += nn;
            }
            int pos = carry + incl - cnt;
            if (mk) s_rank[gi] = (uint16_t)min(pos, 0xffff);  // rank in O of the group's first outlier channel
            while (mk) {
                const int i = __ffs(mk) - 1;
                mk &= mk - 1;
                if (pos < a.cap) {
                    s_oidx[pos] = 8 * gi + i;
                    if (b == 0) a.outlier_idx[pos] = 8 * gi + i;
                }
                ++pos;
            }
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        __syncwarp();
        const int r = min(carry, a.cap);
        // (a.aux_cols == 0: no Aux block and no W_aux wanted, the list of sources has no room and no reader)
        const int ucols = min(crep * r, a.aux_cols);
        for (int i = lane; i < ucols; i += 32) s_auxsrc[i] = (uint16_t)s_oidx[i / crep];
        // own-scale reading, per tensor: max |Aux| = 2^-e times the largest maximum among the listed channels
        float am = 0.0f;
        for (int j = lane; j < r; j += 32) am = fmaxf(am, __uint_as_float(s_colmax[s_oidx[j]]) * down);
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
            __threadfence_block();
            s_list_ready = 1;
        }
        __syncwarp();
        if (kPerToken) __syncthreads();  // the per-token path reads the shared factor copies and the Aux sources
        // W_aux[n, crep*j + i] = W_q[n, O_j]: this CTA's share, one 4-byte word per lane and round.  The GEMM consumes
        // the Aux columns in steps of 32, i.e. columns [0, pad_cols); an Aux column of zeros makes the matching W_aux
        // column irrelevant and vice versa, so both blocks are written up to pad_cols only (codes, then zeros).
        // (With its own scale Aux is the A operand of a product over all aux_cols columns: zeros to the end.)
        if (a.w_aux) {
            const int used_cols = crep * r;
            const int pad_words = a.aux_own ? a.aux_cols >> 2 : ((used_cols + 31) & ~31) >> 2;
            const int total = a.N * pad_words;
            for (int i = b * 32 + lane; i < total; i += gridDim.x * 32) {
                const int n = i / pad_words, w = i - n * pad_words;
                uint32_t packed = 0;
#pragma unroll
                for (int bb = 0; bb < 4; ++bb)
                    if (w * 4 + bb < used_cols)
                        packed |= (uint32_t)(uint8_t)a.w_q[(size_t)n * a.ldw + s_auxsrc[w * 4 + bb]] << (8 * bb);
                *reinterpret_cast<uint32_t *>(a.w_aux + (size_t)n * a.ld_waux + w * 4) = packed;
            }
        }
        if (!kPerToken) {
            // evicted stripes again, newest first: load T + j fetches stripe T - S - 1 - j
            for (int j = 0; j < T - Sres; ++j) {
                if (!issue(T + j, T - Sres - 1 - j)) break;
                issued = T + j + 1;
            }
        }
    } else if (!kPerToken) {
        // -------------------------------------------------------------- pass 2, per-tensor scale
        // The pass-1 mapping again, so the channel factors stay in registers and consecutive lanes store
        // consecutive codes.  Brackets of 1/s with the channel factor folded in (power of two: exact).
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
        // Threads that write Aux bytes (their chunk holds an outlier channel, or they own the last channel group and
        // with it the row's zero padding) need the producer warp's listing: rank of their first outlier channel, r.
        const bool aux_writer = a.aux_q && active && (fmask != 0u || cg == G - 1);
        int my_rank = 0, r = 0;
        float s_aux = 1.0f;
        bool ok = true;
        if (a.aux_q && __any_sync(0xffffffffu, aux_writer)) {
            uint32_t i = 0;
            while (!s_list_ready && ++i < g.spin) { if ((i & 63u) == 63u && *abort_flag) break; }
            ok = __all_sync(0xffffffffu, s_list_ready != 0);
            if (!ok) *abort_flag = 1u;
            r = min(s_r_true, a.cap);
            s_aux = s_aux_scale;
            if (fmask) my_rank = s_rank[cg];
        }
        const int used_cols = crep * r;
        const int pad_cols = a.aux_own ? a.aux_cols : (used_cols + 31) & ~31;
        auto write_aux = [&](const uint4 &v, uint2 code, size_t m) {
            int8_t *arow = a.aux_q + m * a.ld_aux;
            if (fmask) {
                int j = my_rank;
                uint32_t mk = fmask;
                const __half *h = reinterpret_cast<const __half *>(&v);
                while (mk) {
                    const int i = __ffs(mk) - 1;
                    mk &= mk - 1;
                    if (j < a.cap) {
                        int8_t cb;
                        if (a.aux_own) cb = (int8_t)quant_exact(__half2float(h[i]) * down, s_aux, qf);  // Eq. 1, own scale
                        else cb = (int8_t)((i < 4 ? code.x >> (8 * i) : code.y >> (8 * (i - 4))) & 0xffu);
                        for (int rep = 0; rep < crep; ++rep) arow[crep * j + rep] = cb;
                    }
                    ++j;
                }
            }
            if (cg == G - 1)
                for (int col = used_cols; col < pad_cols; ++col) arow[col] = 0;
        };
        const uint8_t *mine = ring + (size_t)row_off * row_bytes + cg * 16;
        for (int q = 0; q < T && ok; ++q) {
            // resident stripes first (load numbers T-Sres .. T-1), then the refetched ones (load T + q - Sres)
            const int n = q < Sres ? T - Sres + q : T + q - Sres;
            const int stripe = q < Sres ? n : T - 1 - q;
            const int slot = n % S;
            if (q >= Sres) {
                ok = wait_warp(&bar_full[slot], (uint32_t)(n / S) & 1u, abort_flag, g.spin);
                if (!ok) break;
            }
            const int row = stripe * nrow + row_off;
            if (active && row < rows) {
                const uint4 v = *reinterpret_cast<const uint4 *>(mine + (size_t)slot * slot_bytes);
                const uint2 cd = codes(v);
                const size_t m = (size_t)r0 + row;
                *reinterpret_cast<uint2 *>(a.body_q + m * a.ld_q + cg * 8) = cd;
                if (aux_writer) write_aux(v, cd, m);
            }
            if (q + Sres < T) {  // a refetch is waiting for this position
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar_empty[slot]);
            }
        }
    }

    if (kPerToken) {
        if (!producer) __syncthreads();  // matches the producer warp's barrier after its listing
        const int r = min(s_r_true, a.cap);
        const int used_cols = crep * r, pad_words = a.aux_own ? a.aux_cols >> 2 : ((used_cols + 31) & ~31) >> 2;
        // where a row lives: the last Sres stripes are resident in the ring, the others are read from global memory
        auto row_src = [&](int row) -> const uint4 * {
            const int stripe = row / nrow;
            if (stripe >= T - Sres)
                return reinterpret_cast<const uint4 *>(ring + (size_t)(stripe % S) * slot_bytes +
                                                       (size_t)(row - stripe * nrow) * row_bytes);
            return reinterpret_cast<const uint4 *>(a.X + ((size_t)r0 + row) * a.ldx);
        };
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
            const uint4 *src = row_src(row);
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

    // ---------------------------------------------------------------- end: status, clean-up for the next call
    __syncthreads();
    if (s_abort) {  // a wait of pass 2 ran out: let the copies in flight land, mark the workspace, leave
        if (producer) drain(issued);
        __syncthreads();
        if (t == 0) {
            atomicOr(&a.ctrl->arrived, kPoisonBit);
            if (a.dev_status) atomicMax(a.dev_status, kStatusTimeout);
        }
        return;
    }
    if (s_last) {
        uint4 *rep4 = reinterpret_cast<uint4 *>(a.colmax_rep);
        for (int i = t; i < kColmaxReplicas * (K >> 2); i += kT) rep4[i] = make_uint4(0u, 0u, 0u, 0u);
        if (t == 0) {
            a.ctrl->arrived = 0u;
            a.ctrl->readers = 0u;
        }
    }
}

}  // namespace

bool prep_supported(int M, int K) { return M >= 1 && K >= 8 && K % 8 == 0 && (K >> 3) <= kMaxG; }

cudaError_t launch_prep(const PrepArgs &a, cudaStream_t s) {
    static const void *const fns[2] = {reinterpret_cast<const void *>(k_prep<false>),
                                       reinterpret_cast<const void *>(k_prep<true>)};
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
    PrepGeom g{};
    g.rows_base = a.M / grid;
    g.rows_extra = a.M % grid;
    const int rows_max = g.rows_base + (g.rows_extra ? 1 : 0);
    const int G = a.K >> 3;
    g.nrow = kConsThreads / G;
    if (g.nrow > rows_max) g.nrow = rows_max;
    const int fixed = fixed_smem_bytes(a.K, a.cap, a.aux_cols);
    const long long slot_bytes = (long long)g.nrow * a.K * 2;
    const int t_max = (rows_max + g.nrow - 1) / g.nrow;
    long long slots = (kMaxDynSmem - fixed) / slot_bytes;
    if (slots > kMaxSlots) slots = kMaxSlots;
    if (slots > t_max) slots = t_max;
    if (slots < 1) return cudaErrorInvalidValue;
    g.slots = (int)slots;
    g.g_magic = ((1u << 20) + (uint32_t)G - 1u) / (uint32_t)G;
    const TestHooks &h = test_hooks();
    g.spin = h.spin_limit ? h.spin_limit : (1u << 22);
    g.extra_arrivals = h.prep_extra_arrivals;
    PrepArgs args = a;
    void *params[] = {&args, &g};
    const void *fn = fns[a.per_token ? 1 : 0];
    return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kT), params, (size_t)(fixed + g.slots * slot_bytes), s);
}

}  // namespace muxq
