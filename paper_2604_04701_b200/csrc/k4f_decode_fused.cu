// K4, fused form: the whole MUXQ layer for M <= 16 token rows in ONE launch -- detection (Section
// III-C), redistribution (Eq. 4-5), quantization (Eq. 1), the INT8 products with the Aux correction
// (Eq. 7) and the dequantization (Eq. 3).  At these sizes the layer is a stream over W_q (N*K bytes)
// and everything else is small, so:
//   prologue  every CTA reads the few rows of X itself (twice, from L2), derives the channel maxima, the
//             outlier flags, the scale(s) and the INT8 codes of X into shared memory -- redundant work
//             per CTA, but no grid-wide barrier, no scratch in global memory and no second launch.
//   stream    a CTA takes 8 output channels at a time; its 16 warps split K into 64-byte segments.
//             A lane loads 16 bytes of one W_q row (8 rows x 64 contiguous bytes per warp load), the
//             matching 16 bytes of X codes come from shared memory, and two mma.sync m16n8k32 (s8 x s8
//             -> s32) consume them.  The K order inside a segment is permuted the same way for both
//             operands (lane q of a row holds bytes 16q..16q+15), which a dot product does not notice.
//             Aux term with the shared scale: Aux_q == Body_q[:, O], so c * sum_{k in O} is a second
//             accumulation with X masked to the outlier channels, issued only for segments that hold one.
//   finish    the 16 partial 16x8 tiles are summed through shared memory, combined as acc_b + c*acc_a
//             (int32, exact), dequantized and stored.
// Tensor-core use here is the small legacy mma.sync form on purpose: the path is bound by the W_q
// stream, and mma.sync needs no TMEM or descriptor set-up for 8-column tiles.
#include "kernels.h"
#include "quant.cuh"

namespace muxq {

namespace {

constexpr int kT = 512;
constexpr int kWarps = kT / 32;
constexpr int kPre = 8;               // 64-byte W segments per warp fetched ahead of the prologue into registers
constexpr int kExtra = 4;             // ... and further ones into shared memory (asynchronous copies)
constexpr int kMaxIter = 2;           // channel groups (8 channels) per thread: K <= 8 * kT * kMaxIter
constexpr int kStatusCapacity = 5;    // MUXQ_ERR_CAPACITY

__device__ __forceinline__ void mma_s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// 16-byte read-only load as a volatile statement: a batch of them is issued back to back before the first use,
// whatever the register allocator would rather do (under register pressure it serialises plain loads).
__device__ __forceinline__ uint4 ld_nc_v4(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

struct Smem {
    int pitch;          // bytes per row of X codes; pitch % 128 == 64 keeps the 8-row x 64-byte reads conflict free
    int off_mask;       // [K] 0xFF at outlier channels
    int off_segflag;    // [K/64] segment holds an outlier channel
    int off_grpmask;    // [K/8] per-group flag bits
    int off_red;        // [2][kWarps][128] int32 partial tiles
    int off_wx;         // [kWarps][kExtra][32] 16-byte pieces of W_q beyond the kPre segments a warp keeps in registers
    int off_xs;         // [MT][K] fp16 copy of X between the two passes (only when it fits), else -1
    int total;
};
constexpr int kMaxSmem = 200 * 1024;
__host__ __device__ inline Smem smem_layout(int MT, int K) {
    Smem s;
    s.pitch = K + ((64 - (K & 127)) & 127);
    if ((s.pitch & 127) != 64) s.pitch += 64;
    s.off_mask = MT * s.pitch;
    s.off_segflag = s.off_mask + K;
    s.off_grpmask = s.off_segflag + (((K >> 6) + 15) & ~15);
    s.off_red = (s.off_grpmask + (K >> 3) + 15) & ~15;
    s.off_wx = s.off_red + 2 * kWarps * 128 * 4;
    s.total = s.off_wx + kWarps * kExtra * 32 * 16;
    s.off_xs = -1;
    if (s.total + MT * K * 2 <= kMaxSmem) {
        s.off_xs = s.total;
        s.total += MT * K * 2;
    }
    return s;
}

// kDotM > 0 (MT == 8, M <= kDotM <= 4): the products are 4-way byte dot products (dp4a) per token row instead of
// mma.sync tiles.  The legacy mma.sync path issues an INT8 m16n8k32 only about every 32 cycles per SM sub-partition
// on this part; for a single row the dot products cost less (measured: 5.3 against 5.7 us per layer at M = 1, but
// 6.8 against 6.2 us at M = 4, so only kDotM = 1 is instantiated).
template <int MT, int kDotM>
__global__ void __launch_bounds__(kT, 1) k_decode_fused(const DecodeFusedArgs a, int tpg) {
    extern __shared__ __align__(16) uint8_t smem[];
    __shared__ uint32_t s_rowmax[16];  // bit patterns of non-negative floats (per-token row maxima of Body)
    __shared__ float s_wmax[kWarps];
    __shared__ float s_rowscale[16];
    __shared__ int s_r;

    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int K = a.K, G = K >> 3, M = a.M;
    const Smem L = smem_layout(MT, K);
    int8_t *xq = reinterpret_cast<int8_t *>(smem);
    uint8_t *s_mask = smem + L.off_mask;
    uint8_t *s_segflag = smem + L.off_segflag;
    uint8_t *s_grpmask = smem + L.off_grpmask;
    int *s_red = reinterpret_cast<int *>(smem + L.off_red);
    uint8_t *xs = L.off_xs >= 0 ? smem + L.off_xs : nullptr;
    uint4 *s_wx = reinterpret_cast<uint4 *>(smem + L.off_wx) + warp * (kExtra * 32) + lane;  // this lane's pieces
    const float down = __int_as_float((127 - a.exp_factor) << 23);  // 2^-e
    const float qf = (float)a.qmax;
    const bool first = blockIdx.x == 0;

    // Let the next kernel in the stream (programmatic dependent launch) become resident as early as there is
    // room for it: it fetches its own weights and then waits for this grid to finish before it touches X or Y.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // The first tile's share of W_q does not depend on X: its loads go out before the prologue, so the
    // HBM latency of the stream overlaps the detection and quantization work.
    const int r = lane >> 2, q = lane & 3;
    const int nseg = K >> 6;
    const int tiles = (a.N + 7) >> 3;
    const int ws = kWarps / tpg;             // warps per team
    const int team = warp / ws;
    // (when tpg does not divide the warp count, the warps left over get no segment: wi = nseg)
    const int wi = team < tpg ? warp - team * ws : nseg;
    uint4 wpre[kPre];
    {
        const int n = (blockIdx.x * tpg + team) * 8 + r;
        const int8_t *wrow = a.w_q + (size_t)min(n, a.N - 1) * a.ldw + q * 16;
#pragma unroll
        for (int u = 0; u < kPre; ++u) {
            const int seg = wi + u * ws;
            wpre[u] = seg < nseg ? __ldg(reinterpret_cast<const uint4 *>(wrow + seg * 64)) : make_uint4(0u, 0u, 0u, 0u);
        }
        // segments beyond kPre (the host allows them only when all groups fit one round): to shared memory
#pragma unroll
        for (int e = 0; e < kExtra; ++e) {
            const int seg = wi + (kPre + e) * ws;
            if (seg < nseg) {
                const uint32_t d = (uint32_t)__cvta_generic_to_shared(s_wx + e * 32);
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(wrow + seg * 64) : "memory");
            }
        }
    }
    const float sw0 = __ldg(a.s_w);  // a constant of the layer like W_q (the per-tensor scale, or the first column's)
    // Everything below reads X or writes results: under programmatic dependent launch it must wait for the
    // kernel before this one in the stream; the weights above are constants and were fetched ahead of that.
    if (t < 16) s_rowmax[t] = 0u;
    for (int i = t; i < (K >> 6); i += kT) s_segflag[i] = 0;
    __syncthreads();  // (shared-memory set-up needs nothing from the predecessor either)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("cp.async.wait_all;" ::: "memory");  // a lane reads back only the pieces it copied itself

    if (first && t == 0 && a.dev_status) *a.dev_status = 0;

    // ---------------------------------------------------------------- pass A: channel maxima, flags, Body maxima
    // The loops over a thread's channel groups are deliberately NOT unrolled: each copy of their bodies would be
    // code this SM has not fetched yet, and instruction fetch is what these short phases wait for.  The groups'
    // outlier flags share one register, a byte per group.
    static_assert(kMaxIter <= 4, "one byte of my_masks per channel group of the thread");
    uint32_t my_masks = 0;
    float bmax = 0.0f;
#pragma unroll 1
    for (int it = 0; it < kMaxIter; ++it) {
        const int cg = t + it * kT;
        if (cg < G) {
            __half2 cm[4];
            cm[0] = cm[1] = cm[2] = cm[3] = __float2half2_rn(0.f);
            for (int m0 = 0; m0 < M; m0 += 4) {  // four independent row loads in flight
                uint4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    v[u] = m0 + u < M ? ld_nc_v4(reinterpret_cast<const uint4 *>(a.X + (size_t)(m0 + u) * a.ldx) + cg)
                                      : make_uint4(0u, 0u, 0u, 0u);
                if (xs) {
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (m0 + u < M) *reinterpret_cast<uint4 *>(xs + (size_t)(m0 + u) * K * 2 + cg * 16) = v[u];
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    cm[0] = __hmax2(cm[0], __habs2(*reinterpret_cast<const __half2 *>(&v[u].x)));
                    cm[1] = __hmax2(cm[1], __habs2(*reinterpret_cast<const __half2 *>(&v[u].y)));
                    cm[2] = __hmax2(cm[2], __habs2(*reinterpret_cast<const __half2 *>(&v[u].z)));
                    cm[3] = __hmax2(cm[3], __habs2(*reinterpret_cast<const __half2 *>(&v[u].w)));
                }
            }
            float c8[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) { c8[2 * i] = __low2float(cm[i]); c8[2 * i + 1] = __high2float(cm[i]); }
            uint32_t mask = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const bool flagged = c8[i] > a.tau;  // strict
                mask |= flagged ? (1u << i) : 0u;
                bmax = fmaxf(bmax, flagged ? c8[i] * down : c8[i]);
            }
            my_masks |= mask << (8 * it);
            s_grpmask[cg] = (uint8_t)mask;
            if (mask) s_segflag[cg >> 3] = 1;
            uint2 mb;
            mb.x = ((mask & 1) ? 0xFFu : 0u) | ((mask & 2) ? 0xFF00u : 0u) | ((mask & 4) ? 0xFF0000u : 0u) |
                   ((mask & 8) ? 0xFF000000u : 0u);
            mb.y = ((mask & 16) ? 0xFFu : 0u) | ((mask & 32) ? 0xFF00u : 0u) | ((mask & 64) ? 0xFF0000u : 0u) |
                   ((mask & 128) ? 0xFF000000u : 0u);
            *reinterpret_cast<uint2 *>(s_mask + cg * 8) = mb;
            if (first && a.colmax) {
                reinterpret_cast<float4 *>(a.colmax)[2 * cg] = make_float4(c8[0], c8[1], c8[2], c8[3]);
                reinterpret_cast<float4 *>(a.colmax)[2 * cg + 1] = make_float4(c8[4], c8[5], c8[6], c8[7]);
            }
        }
    }
    if (a.per_vec) {
        // per-token scales: row maxima of Body (after the 2^-e), a second cheap sweep with the flags known
#pragma unroll 1
        for (int it = 0; it < kMaxIter; ++it) {
            const int cg = t + it * kT;
            if (cg < G) {
                for (int m = 0; m < M; ++m) {
                    const uint4 v = xs ? *reinterpret_cast<const uint4 *>(xs + (size_t)m * K * 2 + cg * 16)
                                       : __ldg(reinterpret_cast<const uint4 *>(a.X + (size_t)m * a.ldx) + cg);
                    float f[8];
                    unpack8(v, f);
                    float rm = 0.0f;
#pragma unroll
                    for (int i = 0; i < 8; ++i) rm = fmaxf(rm, fabsf((my_masks >> (8 * it + i)) & 1u ? f[i] * down : f[i]));
                    if (rm > 0.0f) atomicMax(&s_rowmax[m], __float_as_uint(rm));
                }
            }
        }
    }
    bmax = warp_max(bmax);
    if (lane == 0) s_wmax[warp] = bmax;
    __syncthreads();
    // ---------------------------------------------------------------- scales (Eq. 1)
    if (t < 16) {
        float s;
        if (a.per_vec) {
            const float mx = __uint_as_float(s_rowmax[t]);
            s = mx > 0.0f ? __fdiv_rn(mx, qf) : 1.0f;
            if (first && t < M && a.s_x_rows) a.s_x_rows[t] = s;
        } else {
            float mx = 0.0f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) mx = fmaxf(mx, s_wmax[w]);
            s = mx > 0.0f ? __fdiv_rn(mx, qf) : 1.0f;
            if (first && t == 0 && a.ctrl) { a.ctrl->s_x = s; a.ctrl->inv_s_x = __frcp_rn(s); }
        }
        s_rowscale[t] = s;
    }
    // warp 1 lists O in ascending order for the caller (the products below only need the flags)
    if (warp == 1 && first) {
        int carry = 0;
        for (int base = 0; base < G; base += 32) {
            const int g = base + lane;
            uint32_t m = g < G ? s_grpmask[g] : 0u;
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
                if (pos < a.cap && a.outlier_idx) a.outlier_idx[pos] = 8 * g + i;
                ++pos;
            }
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) {
            if (a.ctrl) a.ctrl->n_outliers = carry;
            if (carry > a.cap && a.dev_status) atomicMax(a.dev_status, kStatusCapacity);
        }
    }
    if (warp == 2) {  // every CTA needs r only to know whether the capacity was exceeded
        int cnt = 0;
        for (int g = lane; g < G; g += 32) cnt += __popc((uint32_t)s_grpmask[g]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        if (lane == 0) s_r = cnt;
    }
    __syncthreads();

    // ---------------------------------------------------------------- pass B: codes of X into shared memory
    // Work items are (channel group, batch of four rows), spread over all threads: with one thread per channel group
    // the rows would be walked one after the other by a fraction of the CTA.  The flags come from shared memory.
    {
        float lo = 0.0f, hi = 0.0f;
        if (!a.per_vec) recip_bracket(__frcp_rn(s_rowscale[0]), lo, hi);
#pragma unroll 1
        for (int item = t; item < G * (MT / 4); item += kT) {
            const int batch = item / G, cg = item - batch * G, m0 = 4 * batch;
            const uint32_t gmask = s_grpmask[cg];
            float mul[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) mul[i] = (gmask >> i) & 1u ? down : 1.0f;
            uint4 v[4];  // four independent row loads in flight
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                v[u] = make_uint4(0u, 0u, 0u, 0u);
                if (m0 + u < M)
                    v[u] = xs ? *reinterpret_cast<const uint4 *>(xs + (size_t)(m0 + u) * K * 2 + cg * 16)
                              : ld_nc_v4(reinterpret_cast<const uint4 *>(a.X + (size_t)(m0 + u) * a.ldx) + cg);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int m = m0 + u;
                uint2 code = make_uint2(0u, 0u);
                if (m < M) {
                    float f[8];
                    unpack8(v[u], f);
#pragma unroll
                    for (int i = 0; i < 8; ++i) f[i] *= mul[i];  // exact
                    const float s = s_rowscale[a.per_vec ? m : 0];
                    if (a.per_vec) recip_bracket(__frcp_rn(s), lo, hi);
                    // the scale comes from these very values: no code can leave the range (bracket form)
                    uint32_t cb[8];
                    if (quant8_bracket(f, lo, hi, cb)) code = codes_exact(v[u], gmask, down, s, qf);  // rare
                    else code = pack8(cb);
                }
                *reinterpret_cast<uint2 *>(xq + m * L.pitch + cg * 8) = code;
            }
        }
    }
    __syncthreads();
    if (s_r > a.cap) return;  // MUXQ_ERR_CAPACITY was raised; Y is unspecified

    // ---------------------------------------------------------------- stream W_q
    // A CTA works on a group of tpg 8-channel tiles at a time; team j of its warps takes tile j of the
    // group and splits K among its members, so that every lane keeps several 16-byte loads in flight
    // whatever K is.
    const int groups = (tiles + tpg - 1) / tpg;
    for (int group = blockIdx.x; group < groups; group += gridDim.x) {
        const int8_t *xlo = xq + r * L.pitch + q * 16;
        // two Body accumulators (the two halves of a 64-byte segment): consecutive mma.sync on one accumulator
        // wait for each other
        int accb[4] = {0, 0, 0, 0}, accb2[4] = {0, 0, 0, 0}, acca[4] = {0, 0, 0, 0};
        auto consume = [&](int seg, const uint4 &w) {
            if constexpr (kDotM > 0) {
                // lane (r, q) holds 16 bytes of W_q row r; the same 16 channels of token row m come from shared memory
                // (the 8 lanes with equal q read one address).  accb[m] / acca[m]: Body and Aux sums of row m.
                const bool fl = s_segflag[seg] != 0;  // warp-uniform
                uint4 mk = make_uint4(0u, 0u, 0u, 0u);
                if (fl) mk = *reinterpret_cast<const uint4 *>(s_mask + seg * 64 + q * 16);
#pragma unroll
                for (int m = 0; m < kDotM; ++m) {
                    const uint4 x = *reinterpret_cast<const uint4 *>(xq + m * L.pitch + q * 16 + seg * 64);
                    accb[m] = __dp4a((int)w.x, (int)x.x, accb[m]);
                    accb[m] = __dp4a((int)w.y, (int)x.y, accb[m]);
                    accb[m] = __dp4a((int)w.z, (int)x.z, accb[m]);
                    accb[m] = __dp4a((int)w.w, (int)x.w, accb[m]);
                    if (fl) {
                        acca[m] = __dp4a((int)w.x, (int)(x.x & mk.x), acca[m]);
                        acca[m] = __dp4a((int)w.y, (int)(x.y & mk.y), acca[m]);
                        acca[m] = __dp4a((int)w.z, (int)(x.z & mk.z), acca[m]);
                        acca[m] = __dp4a((int)w.w, (int)(x.w & mk.w), acca[m]);
                    }
                }
                return;
            }
            const uint4 alo = *reinterpret_cast<const uint4 *>(xlo + seg * 64);
            uint4 ahi = make_uint4(0u, 0u, 0u, 0u);
            if (MT == 16) ahi = *reinterpret_cast<const uint4 *>(xlo + 8 * L.pitch + seg * 64);
            mma_s8(accb, alo.x, ahi.x, alo.y, ahi.y, w.x, w.y);
            mma_s8(accb2, alo.z, ahi.z, alo.w, ahi.w, w.z, w.w);
            if (s_segflag[seg]) {  // warp-uniform: Aux term on the outlier channels of this segment
                const uint4 mk = *reinterpret_cast<const uint4 *>(s_mask + seg * 64 + q * 16);
                mma_s8(acca, alo.x & mk.x, ahi.x & mk.x, alo.y & mk.y, ahi.y & mk.y, w.x, w.y);
                mma_s8(acca, alo.z & mk.z, ahi.z & mk.z, alo.w & mk.w, ahi.w & mk.w, w.z, w.w);
            }
        };
        // this warp's first kPre segments are already in registers
#pragma unroll
        for (int u = 0; u < kPre; ++u) {
            const int seg = wi + u * ws;
            if (seg < nseg) consume(seg, wpre[u]);
        }
        // the others: from shared memory for the CTA's first group, else straight from global memory
#pragma unroll 1
        for (int e = 0; e < kExtra; ++e) {
            const int seg = wi + (kPre + e) * ws;
            if (seg >= nseg) break;
            uint4 w;
            if (group == (int)blockIdx.x) {
                w = s_wx[e * 32];
            } else {
                const int n = (group * tpg + team) * 8 + r;
                w = __ldg(reinterpret_cast<const uint4 *>(a.w_q + (size_t)min(n, a.N - 1) * a.ldw + q * 16 + seg * 64));
            }
            consume(seg, w);
        }
        // fetch the next group's segments now; they arrive while this group is reduced and stored
        if (group + (int)gridDim.x < groups) {
            const int nn0 = ((group + gridDim.x) * tpg + team) * 8;
            const int8_t *wnext = a.w_q + (size_t)min(nn0 + r, a.N - 1) * a.ldw + q * 16;
#pragma unroll
            for (int u = 0; u < kPre; ++u) {
                const int seg = wi + u * ws;
                if (seg < nseg) wpre[u] = __ldg(reinterpret_cast<const uint4 *>(wnext + seg * 64));
            }
        }
        // acc = acc_b + c * acc_a (Eq. 7), partial over this warp's K segments; element (row, col) of the
        // 16 x 8 tile: this lane holds rows r and r+8, columns 2q and 2q+1
        int *red = s_red + warp * 128;
        if constexpr (kDotM > 0) {
            // the four lanes of a W_q row add up; rows >= kDotM of the 16 x 8 tile are never stored (m < M below)
#pragma unroll
            for (int m = 0; m < kDotM; ++m) {
                int v = accb[m] + a.c * acca[m];
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                if (q == 0) red[m * 8 + r] = v;
            }
        } else {
            red[r * 8 + 2 * q] = accb[0] + accb2[0] + a.c * acca[0];
            red[r * 8 + 2 * q + 1] = accb[1] + accb2[1] + a.c * acca[1];
            red[(r + 8) * 8 + 2 * q] = accb[2] + accb2[2] + a.c * acca[2];
            red[(r + 8) * 8 + 2 * q + 1] = accb[3] + accb2[3] + a.c * acca[3];
        }
        __syncthreads();
        for (int e = t; e < 128 * tpg; e += kT) {
            const int j = e >> 7, el = e & 127;  // tile of the group, element of its 16 x 8 tile
            int acc = 0;
            for (int w = 0; w < ws; ++w) acc += s_red[(j * ws + w) * 128 + el];
            const int m = el >> 3, nn = (group * tpg + j) * 8 + (el & 7);
            if (m < M && nn < a.N) {
                const size_t o = (size_t)m * a.ldy + nn;
                if (a.out_kind == 2) {
                    reinterpret_cast<int32_t *>(a.Y)[o] = acc;
                } else {
                    const float sx = s_rowscale[a.per_vec ? m : 0];
                    const float sw = a.per_vec ? __ldg(a.s_w + nn) : sw0;
                    float y = __fmul_rn(__fmul_rn(sx, sw), __int2float_rn(acc));  // Eq. 3
                    if (a.bias) y = __fadd_rn(y, __ldg(a.bias + nn));
                    if (a.out_kind == 1) reinterpret_cast<float *>(a.Y)[o] = y;
                    else reinterpret_cast<__half *>(a.Y)[o] = __float2half_rn(y);
                }
            }
        }
        __syncthreads();
    }
}

}  // namespace

bool decode_fused_supported(int M, int K) { return M >= 1 && M <= 16 && K % 64 == 0 && K <= 8 * kT * kMaxIter; }

cudaError_t launch_decode_fused(const DecodeFusedArgs &a, cudaStream_t s) {
    const int MT = a.M <= 8 ? 8 : 16;
    const Smem L = smem_layout(MT, a.K);
    static bool attr_set = false;
    if (!attr_set) {
        const void *fns[3] = {reinterpret_cast<const void *>(k_decode_fused<8, 1>),
                              reinterpret_cast<const void *>(k_decode_fused<8, 0>),
                              reinterpret_cast<const void *>(k_decode_fused<16, 0>)};
        for (const void *f : fns) {
            cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
            if (e != cudaSuccess) return e;
        }
        attr_set = true;
    }
    if (L.total > kMaxSmem) return cudaErrorInvalidValue;
    // tiles per group: the smallest power of two that gives every warp at least 4 segments of 64 bytes
    const int nseg = a.K / 64, tiles = (a.N + 7) / 8;
    // A warp holds kPre segments in registers and up to kExtra more in shared memory; the latter only pays when it
    // saves a round of groups over the SMs (a second round costs a CTA a whole extra stream-and-reduce latency).
    // Order of preference: fewest rounds; all segments in registers; at least 4 segments per warp; fewest tiles.
    int tpg = 1;
    {
        long best = -1;
        for (int T = 1; T <= kWarps; ++T) {
            const int wsT = kWarps / T, spw = (nseg + wsT - 1) / wsT;
            const int g = (tiles + T - 1) / T, rounds = (g + num_sms() - 1) / num_sms();
            if (spw > kPre + kExtra || (spw > kPre && rounds > 1)) continue;
            const long key = ((long)rounds << 24) | ((spw > kPre ? 1L : 0L) << 16) | ((spw >= 4 ? 0L : 1L) << 8) | T;
            if (best < 0 || key < best) { best = key; tpg = T; }
        }
    }
    const int groups = (tiles + tpg - 1) / tpg;
    // at most one CTA per SM, so that the kernel of the next layer in the stream can become resident beside
    // this one (programmatic dependent launch) and fetch its weights while this one finishes
    int grid = num_sms();
    if (grid > groups) grid = groups;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kT);
    cfg.dynamicSmemBytes = (size_t)L.total;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    if (a.M == 1) return cudaLaunchKernelEx(&cfg, k_decode_fused<8, 1>, a, tpg);
    if (MT == 8) return cudaLaunchKernelEx(&cfg, k_decode_fused<8, 0>, a, tpg);
    return cudaLaunchKernelEx(&cfg, k_decode_fused<16, 0>, a, tpg);
}

}  // namespace muxq
