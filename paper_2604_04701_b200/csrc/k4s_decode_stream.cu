// K4, streaming form: one persistent launch that walks a list of decode-shaped MUXQ layers (M <= 16 token rows
// each; Section III-C, Eq. 1, Eq. 4-5, Eq. 7, Eq. 3 per layer, exactly as the one-layer decode kernel computes
// them).  At these sizes a layer is a stream over its W_q (N*K bytes) and little else, and one launch per layer
// cannot keep HBM busy: a layer moves 1.6-6.6 MB, less than a microsecond of HBM time.  Here the weight stream
// never stops at a layer boundary:
//   loader warps    walk the list of layers and, for every unit of 8 output channels that belongs to this CTA,
//                   fetch the 8 rows of W_q with bulk asynchronous copies (cp.async.bulk, no multicast) into a
//                   ring of shared-memory stages; the copies report their bytes to the stage's mbarrier.  They
//                   depend on nothing but the ring's free slots, so they run several layers ahead of the
//                   arithmetic.  Each loader warp takes every fourth stage on its own: one loop over the stages
//                   (wait for the slot, issue, next) costs a single warp several hundred cycles per stage however
//                   the bytes are moved (measured: 10 KB per 0.3 us, 4.4 TB/s over 148 SMs, with one loop of 128
//                   threads making 16-byte copies; 6.7-7 TB/s with four independent loops), and with one bulk
//                   copy per stage or per row the loop is a few dozen instructions.
//   prepare warps   per layer: derive the channel maxima, the outlier flags, the scale(s) and the INT8 codes of X
//                   into a shared-memory buffer (redundant per CTA, no grid-wide exchange).  The phases of one
//                   layer are short serial chains with barriers in between, so for small M several groups of
//                   warps work on different layers at once (one buffer more than groups), and the fp16 rows
//                   of X are fetched a layer ahead with asynchronous copies.
//   unit warps      per layer: each unit is taken by ONE warp, which accumulates the unit's 8 x M outputs over all
//                   of K in registers (4-way byte dot products for M <= 4, mma.sync m16n8k32 above), adds the Aux
//                   term of Eq. 7 for the 64-byte segments that hold an outlier channel, dequantizes and stores.
// Units go to CTAs round-robin with an offset that keeps running from layer to layer, so that the bytes a CTA
// streams even out over a few layers although a single layer rarely divides evenly.
// Layers are independent unless a layer's flags say that its X is written by the layer before it: then the
// prepare warps first wait for this CTA's unit warps to finish that layer and pass a bounded grid-wide barrier
// (the launch is cooperative); the loaders do not wait.
// All waits are bounded; a wait that runs out raises MUXQ_ERR_TIMEOUT and every role leaves.
#include <mutex>

#include "kernels.h"
#include "ptx.cuh"
#include "quant.cuh"

namespace muxq {

namespace {

constexpr int kUW = 8;                  // unit warps (warps 0..7)
constexpr int kPW = 8;                  // prepare warps (warps 8..15)
constexpr int kLW = 4;                  // loader warps (warps 16..19)
constexpr int kLoader0 = kUW + kPW;     // index of the first loader warp
constexpr int kThreads = 32 * (kLoader0 + kLW);
constexpr int kMaxK = 8192;             // widest layer: 1024 channel groups of 8
constexpr int kMaxGroups = 4;           // groups of prepare warps, each on a layer of its own
constexpr int kMaxBufs = kMaxGroups + 1;
constexpr int kMaxSlots = 24;
constexpr int kStatusCapacity = 5;      // MUXQ_ERR_CAPACITY
constexpr int kStatusTimeout = 6;       // MUXQ_ERR_TIMEOUT
constexpr int kMaxSmem = 227 * 1024 - 1024;

__device__ __forceinline__ void mma_s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// 16 bytes global -> shared, asynchronously (the fp16 rows of X; completion through cp.async.wait_all)
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
// `bytes` (a multiple of 16, both addresses 16-byte aligned) global -> shared by the copy engine; the bytes are
// reported to the mbarrier as they land
__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gsrc, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// Bounded wait of a whole converged warp that backs off between polls: the warps of this kernel spend most of
// their time waiting for each other, and a warp that polls without pause takes issue slots from the few that work.
__device__ __forceinline__ bool wait_sleep(uint64_t *bar, uint32_t parity, volatile uint32_t *abort_flag, uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i) {
        if (__any_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
        if (i >= 2) __nanosleep(i < 16 ? 40 : 200);
        if ((i & 15u) == 15u && __any_sync(0xffffffffu, *abort_flag != 0u)) return false;
    }
    *abort_flag = 1u;
    return false;
}

// named barrier `id` over `nthreads` threads (one per group of prepare warps)
__device__ __forceinline__ void bar_prep(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
// the same barrier, which also tells every one of its threads whether any of them has seen `flag`
__device__ __forceinline__ bool bar_prep_or(int id, int nthreads, bool flag) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, %2, %3, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}\n"
        : "=r"(r)
        : "r"((uint32_t)flag), "r"(id), "r"(nthreads)
        : "memory");
    return r != 0;
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// A buffer that holds a layer's prepared X (sized for the widest K of the list).
struct XLayout {
    int pitch;          // bytes per row of X codes; pitch % 128 == 64 keeps the 8-row x 64-byte reads conflict free
    int off_xq;         // [rows][pitch] INT8 codes (behind a 128-byte header: 16 row scales, r, list length)
    int off_mask;       // [K] 0xFF at outlier channels
    int off_segflag;    // [K/64] segment holds an outlier channel
    int off_grpmask;    // [K/8] per-group flag bits
    int off_flaglist;   // [K/64] u16: the segments that hold an outlier channel, ascending
    int buf_bytes;
    int xs_bytes;       // bytes of one fp16 staging copy of X ([M][K]); 0 when X is not staged
    int total;          // the buffers + two staging copies per group of prepare warps
};
__host__ __device__ inline XLayout x_layout(int rows, int M, int K, bool stage_x, int nbuf, int groups) {
    XLayout s;
    s.pitch = K + ((64 - (K & 127)) & 127);
    if ((s.pitch & 127) != 64) s.pitch += 64;
    s.off_xq = 128;
    s.off_mask = s.off_xq + rows * s.pitch;
    s.off_segflag = s.off_mask + K;
    s.off_grpmask = s.off_segflag + (((K >> 6) + 15) & ~15);
    s.off_flaglist = (s.off_grpmask + (K >> 3) + 15) & ~15;
    s.buf_bytes = (s.off_flaglist + 2 * (K >> 6) + 127) & ~127;
    s.xs_bytes = stage_x ? M * K * 2 : 0;
    s.total = nbuf * s.buf_bytes + 2 * groups * s.xs_bytes;
    return s;
}
struct XHeader {        // first bytes of a buffer
    float rowscale[16];
    int r;              // outlier channels of this layer's X
    int nflag;          // entries of the list of flagged segments
};

struct RingPos {
    int slot;
    uint32_t use;
    __device__ __forceinline__ void advance(int n, int S) {  // n < 2 * S
        slot += n;
        while (slot >= S) { slot -= S; ++use; }
    }
};

// MT: token rows padded to 8 or 16.  kDotM > 0 (M <= kDotM <= 4): products as 4-way byte dot products per token row;
// kDotM == 0: mma.sync tiles of 16 token rows x 8 output channels.
template <int MT, int kDotM>
__global__ void __launch_bounds__(kThreads, 1) k_decode_stream(const ChainArgs a) {
    constexpr int kRows = kDotM > 0 ? kDotM : MT;  // rows of codes a buffer holds
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ uint64_t bar_full[kMaxSlots], bar_empty[kMaxSlots];
    __shared__ uint64_t bar_ready[kMaxBufs], bar_free[kMaxBufs];  // a buffer of prepared X: filled / no longer read
    __shared__ uint32_t s_rowmax[kMaxGroups][16];   // bit patterns of non-negative floats (row maxima of Body)
    __shared__ float s_wmax[kPW];
    __shared__ uint32_t s_abort;
    __shared__ volatile uint32_t s_begun[kMaxSlots];  // uses of a slot the loaders have begun to fill so far

    const int t = threadIdx.x, lane = t & 31;
    const int warp = __shfl_sync(0xffffffffu, t >> 5, 0);  // warp-uniform by construction
    const int S = a.slots, M = a.M, NB = a.nbuf, PG = a.pgroups;
    const int grid = (int)gridDim.x, cta = (int)blockIdx.x;
    uint8_t *ring = smem;
    ChainLayer *tab = reinterpret_cast<ChainLayer *>(smem + (size_t)S * a.slot_bytes);
    uint8_t *xbase = reinterpret_cast<uint8_t *>(tab + a.n_layers);
    const XLayout L = x_layout(kRows, M, a.kmax, a.stage_x != 0, NB, PG);
    volatile uint32_t *abort_flag = &s_abort;

    // the layer table into shared memory (16-byte pieces), barriers
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(a.layers);
        uint4 *dst = reinterpret_cast<uint4 *>(tab);
        for (int i = t; i < a.n_layers * 4; i += kThreads) dst[i] = __ldg(src + i);
    }
    if (t == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&bar_full[s], 1);    // the loader's arrival that announces the stage's bytes; the copies report them
            mbar_init(&bar_empty[s], 1);   // the one unit warp that took the stage
            s_begun[s] = 0u;
        }
        for (int b = 0; b < kMaxBufs; ++b) {
            mbar_init(&bar_ready[b], 1);   // one prepare thread, after its group's barrier
            mbar_init(&bar_free[b], kUW);  // every unit warp, once per layer
        }
        s_abort = 0u;
        fence_barrier_init();
    }
    __syncthreads();

    // the units of a layer that belong to this CTA: first, first + grid, ... below N / 8
    auto first_unit = [&](const ChainLayer &ly) {
        int f = cta - ly.unit_off;
        if (f < 0) f += grid;
        return f;
    };

    if (warp >= kLoader0) {
        // ------------------------------------------------------------ loaders: W_q of every layer, in order.
        // The weights are constants of the layers: nothing here waits for X or a barrier.  Loader warp g fills
        // the stages of this CTA whose running number is g modulo the number of loader warps in use, which
        // divides the number of slots: a slot is always refilled by the warp that filled it before (a warp that
        // met another warp's slot could mistake an older phase of its barrier).
        // A stage is 8 rows of `seg` bytes, stored row after row: one copy when the rows are contiguous in W_q
        // (seg == K == ldw), else one copy per row, issued by 8 lanes.
        const int wl = warp - kLoader0, LG = a.lgroups;
        uint32_t lseq = 0;  // number of this CTA's stages before the current layer
        bool ok = wl < LG;
        for (int l = 0; l < a.n_layers && ok; ++l) {
            const ChainLayer ly = tab[l];
            const int units = ly.N >> 3, nst = ly.K / ly.seg;
            const int first = first_unit(ly);
            const int cnt = first < units ? (units - first + grid - 1) / grid : 0;
            const uint32_t nstage = (uint32_t)(cnt * nst);
            const bool flat = ly.seg == ly.ldw;
            uint32_t j = (uint32_t)(wl + LG - (int)(lseq % (uint32_t)LG)) % (uint32_t)LG;  // first stage of the layer that is this warp's
            int i = (int)j / nst, st = (int)j - i * nst;                                    // its unit and K slice
            for (; j < nstage; j += LG) {
                const uint32_t seq = lseq + j;
                const int slot = (int)(seq % (uint32_t)S);
                const uint32_t use = seq / (uint32_t)S;
                if (use > 0 && !wait_sleep(&bar_empty[slot], (use - 1u) & 1u, abort_flag, a.spin)) {
                    ok = false;
                    break;
                }
                uint8_t *dst = ring + (size_t)slot * a.slot_bytes;
                const int8_t *src = ly.w_q + (size_t)(first + i * grid) * 8 * ly.ldw + (size_t)st * ly.seg;
                if (lane == 0) {
                    s_begun[slot] = use + 1u;  // the slot's previous use is over: its barrier may be waited on
                    mbar_expect_tx(&bar_full[slot], 8u * (uint32_t)ly.seg);
                }
                __syncwarp();
                if (flat) {
                    if (lane == 0) bulk_load(dst, src, 8u * (uint32_t)ly.seg, &bar_full[slot]);
                } else if (lane < 8) {
                    bulk_load(dst + lane * ly.seg, src + (size_t)lane * ly.ldw, (uint32_t)ly.seg, &bar_full[slot]);
                }
                st += LG;
                while (st >= nst) { st -= nst; ++i; }
            }
            lseq += nstage;
        }
        // This warp leaves only when the copies it has issued have landed (they all have when the list was walked
        // to its end, since a unit warp has waited for each; after a time-out some may still be on their way).
        if (wl < LG)
            for (int slot = wl; slot < S; slot += LG) {
                const uint32_t begun = s_begun[slot];
                if (begun > 0u) {
                    bool landed = false;
                    for (uint32_t k = 0; k < a.spin && !landed; ++k) landed = mbar_try_wait(&bar_full[slot], (begun - 1u) & 1u);
                }
            }
    } else if (warp >= kUW) {
        // ------------------------------------------------------------ prepare warps: X of layer l into buffer l mod NB
        // PG groups of warps.  Layer l belongs to group (l + l / PG) mod PG: every run of PG consecutive layers gives
        // each group one layer, and the assignment shifts by one from run to run, so that a list with a period of
        // PG layers (the four projections of a block) does not hand the same group the widest layer every time.
        const int wp = warp - kUW, wpg = kPW / PG, gi = wp / wpg, wg = wp - gi * wpg;
        const int GT = 32 * wpg, tp = t - 32 * (kUW + gi * wpg), bid = 1 + gi;
        const float down = __int_as_float((127 - a.exp_factor) << 23);  // 2^-e
        const float qf = (float)a.qmax;
        const bool first_cta = cta == 0;
        uint32_t *rowmax = s_rowmax[gi];
        // asynchronous copy of the fp16 rows of a layer's X into one of this group's two staging copies
        auto group_of = [&](int l) { return (l + l / PG) % PG; };
        auto next_mine = [&](int l) {  // the next layer of this group behind layer l (or n_layers)
            for (++l; l < a.n_layers && group_of(l) != gi; ++l) {}
            return l;
        };
        auto stage_x = [&](int l, int copy) {
            const ChainLayer &ly = tab[l];
            uint8_t *dst = xbase + NB * L.buf_bytes + (2 * gi + copy) * L.xs_bytes;
            const int G = ly.K >> 3;
            for (int cg = tp; cg < G; cg += GT)
                for (int m = 0; m < M; ++m) cp_async16(dst + (size_t)m * ly.K * 2 + cg * 16, ly.X + (size_t)m * ly.ldx + cg * 8);
        };
        const bool staged = L.xs_bytes > 0;
        auto waits_for_prev = [&](int l) { return (tab[l].flags & kChainWaitPrev) && a.barrier; };
        int mine = 0;  // layers this group has prepared so far: parity selects the staging copy
        {
            const int l0 = next_mine(-1);
            if (staged && l0 < a.n_layers && !waits_for_prev(l0)) stage_x(l0, 0);
        }
        bool stop = false;
        for (int l = next_mine(-1); l < a.n_layers && !stop; l = next_mine(l), ++mine) {
            const ChainLayer ly = tab[l];
            const int K = ly.K, G = K >> 3, b = l % NB, ph = l / NB;
            uint8_t *buf = xbase + b * L.buf_bytes;
            XHeader *hdr = reinterpret_cast<XHeader *>(buf);
            int8_t *xq = reinterpret_cast<int8_t *>(buf + L.off_xq);
            uint8_t *s_mask = buf + L.off_mask, *s_segflag = buf + L.off_segflag, *s_grpmask = buf + L.off_grpmask;
            const uint8_t *xs = staged ? xbase + NB * L.buf_bytes + (2 * gi + (mine & 1)) * L.xs_bytes : nullptr;
            const bool wait_prev = waits_for_prev(l);
            bool ok = true;
            // the buffer was last read for layer l - NB
            if (l >= NB) ok = wait_sleep(&bar_free[b], (uint32_t)(ph - 1) & 1u, abort_flag, a.spin);
            if (wait_prev) {
                // X of this layer is Y of the layer before it: this CTA's unit warps must have stored theirs (they
                // arrive on the buffer's barrier after their stores), then every CTA's must be visible.  The flags
                // carry the ordinal of this wait, which gives the arrival count to wait for.
                ok = ok && wait_sleep(&bar_free[(l - 1) % NB], (uint32_t)((l - 1) / NB) & 1u, abort_flag, a.spin);
                bar_prep(bid, GT);
                if (tp == 0) {
                    __threadfence();
                    atomicAdd(a.barrier, 1u);
                    const uint32_t want = (uint32_t)(ly.flags >> 1) * (uint32_t)grid;
                    bool seen = false;
                    for (uint32_t i = 0; i < a.spin; ++i)
                        if (ld_acquire_u32(a.barrier) >= want) { seen = true; break; }
                    if (!seen) *abort_flag = 1u;
                }
                bar_prep(bid, GT);
                if (staged) stage_x(l, mine & 1);  // could not be fetched ahead
            }
            if (tp < 16) rowmax[tp] = 0u;
            for (int i = tp; i < (K >> 6); i += GT) s_segflag[i] = 0;
            if (staged) asm volatile("cp.async.wait_all;" ::: "memory");
            bar_prep(bid, GT);  // this layer's staging copy is complete and visible; the group's other copy is free
            {
                const int ln = next_mine(l);
                if (staged && ln < a.n_layers && !waits_for_prev(ln)) stage_x(ln, (mine + 1) & 1);
            }
            auto x_chunk = [&](int m, int cg) -> uint4 {
                return xs ? *reinterpret_cast<const uint4 *>(xs + (size_t)m * K * 2 + cg * 16)
                          : __ldcg(reinterpret_cast<const uint4 *>(ly.X + (size_t)m * ly.ldx) + cg);
            };

            // ---------------------------------------------------------- pass A: channel maxima, flags, Body maxima
            float bmax = 0.0f;
#pragma unroll 2
            for (int cg = tp; cg < G; cg += GT) {
                __half2 cm[4];
                cm[0] = cm[1] = cm[2] = cm[3] = __float2half2_rn(0.f);
                for (int m0 = 0; m0 < M; m0 += 4) {  // four independent row loads in flight
                    uint4 v[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) v[u] = m0 + u < M ? x_chunk(m0 + u, cg) : make_uint4(0u, 0u, 0u, 0u);
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
                s_grpmask[cg] = (uint8_t)mask;
                if (mask) s_segflag[cg >> 3] = 1;
                uint2 mb;
                mb.x = ((mask & 1) ? 0xFFu : 0u) | ((mask & 2) ? 0xFF00u : 0u) | ((mask & 4) ? 0xFF0000u : 0u) |
                       ((mask & 8) ? 0xFF000000u : 0u);
                mb.y = ((mask & 16) ? 0xFFu : 0u) | ((mask & 32) ? 0xFF00u : 0u) | ((mask & 64) ? 0xFF0000u : 0u) |
                       ((mask & 128) ? 0xFF000000u : 0u);
                *reinterpret_cast<uint2 *>(s_mask + cg * 8) = mb;
            }
            if (a.per_vec) {
                // per-token scales: row maxima of Body (after the 2^-e), a second cheap sweep with the flags known
#pragma unroll 1
                for (int cg = tp; cg < G; cg += GT) {
                    const uint32_t gmask = s_grpmask[cg];  // this thread's own store
                    for (int m = 0; m < M; ++m) {
                        float f[8];
                        unpack8(x_chunk(m, cg), f);
                        float rm = 0.0f;
#pragma unroll
                        for (int i = 0; i < 8; ++i) rm = fmaxf(rm, fabsf((gmask >> i) & 1u ? f[i] * down : f[i]));
                        if (rm > 0.0f) atomicMax(&rowmax[m], __float_as_uint(rm));
                    }
                }
            }
            bmax = warp_max(bmax);
            if (lane == 0) s_wmax[wp] = bmax;
            bar_prep(bid, GT);
            // ---------------------------------------------------------- scales (Eq. 1), outlier count, flagged segments
            if (tp < 16) {
                float sc;
                if (a.per_vec) {
                    const float mx = __uint_as_float(rowmax[tp]);
                    sc = mx > 0.0f ? __fdiv_rn(mx, qf) : 1.0f;
                } else {
                    float mx = 0.0f;
                    for (int w = 0; w < wpg; ++w) mx = fmaxf(mx, s_wmax[gi * wpg + w]);
                    sc = mx > 0.0f ? __fdiv_rn(mx, qf) : 1.0f;
                }
                hdr->rowscale[tp] = sc;
            }
            if (wg == wpg - 1) {
                int cnt = 0;
                for (int gj = lane; gj < G; gj += 32) cnt += __popc((uint32_t)s_grpmask[gj]);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
                if (lane == 0) {
                    hdr->r = cnt;
                    if (cnt > a.cap && first_cta && a.dev_status) atomicMax(a.dev_status, kStatusCapacity);
                }
                // the flagged 64-byte segments, compacted in ascending order
                uint16_t *flaglist = reinterpret_cast<uint16_t *>(buf + L.off_flaglist);
                int nf = 0;
                for (int base = 0; base < (K >> 6); base += 32) {
                    const bool f = base + lane < (K >> 6) && s_segflag[base + lane] != 0;
                    const uint32_t bal = __ballot_sync(0xffffffffu, f);
                    if (f) flaglist[nf + __popc(bal & ((1u << lane) - 1u))] = (uint16_t)(base + lane);
                    nf += __popc(bal);
                }
                if (lane == 0) hdr->nflag = nf;
            }
            bar_prep(bid, GT);
            const int r = hdr->r;
            if (first_cta && tp == 0 && a.results) {
                ChainResult rr;
                rr.n_outliers = r;
                rr.status = r > a.cap ? kStatusCapacity : 0;
                rr.s_x = hdr->rowscale[0];
                rr.reserved = 0;
                a.results[l] = rr;
            }
            // ---------------------------------------------------------- pass B: codes of X into the buffer
            // (r beyond the capacity: Y of this layer is unspecified, no codes are needed)
            if (r <= a.cap) {
                float lo = 0.0f, hi = 0.0f;
                if (!a.per_vec) recip_bracket(__frcp_rn(hdr->rowscale[0]), lo, hi);
                // items = channel group x batch of four rows
                constexpr int kBatches = kRows / 4 > 0 ? kRows / 4 : 1;
#pragma unroll 2
                for (int item = tp; item < G * kBatches; item += GT) {
                    int batch = 0, cg = item;
                    if (kBatches > 1) { batch = item / G; cg = item - batch * G; }
                    const int m0 = 4 * batch;
                    const uint32_t gmask = s_grpmask[cg];
                    float mul[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) mul[i] = (gmask >> i) & 1u ? down : 1.0f;
                    uint4 v[4];  // four independent row loads in flight
#pragma unroll
                    for (int u = 0; u < 4; ++u) v[u] = (u < kRows && m0 + u < M) ? x_chunk(m0 + u, cg) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int m = m0 + u;
                        if (u >= kRows) break;
                        uint2 code = make_uint2(0u, 0u);
                        if (m < M) {
                            float f[8];
                            unpack8(v[u], f);
#pragma unroll
                            for (int i = 0; i < 8; ++i) f[i] *= mul[i];  // exact
                            const float sc = hdr->rowscale[a.per_vec ? m : 0];
                            if (a.per_vec) recip_bracket(__frcp_rn(sc), lo, hi);
                            uint32_t cb[8];
                            if (quant8_bracket(f, lo, hi, cb)) code = codes_exact(v[u], gmask, down, sc, qf);  // rare
                            else code = pack8(cb);
                        }
                        *reinterpret_cast<uint2 *>(xq + m * L.pitch + cg * 8) = code;
                    }
                }
            }
            // every prepare thread's writes are ordered before the one arrival that hands the buffer to the unit warps
            stop = bar_prep_or(bid, GT, !ok || *abort_flag != 0u);
            if (tp == 0 && !stop) mbar_arrive(&bar_ready[b]);
        }
    } else {
        // ------------------------------------------------------------ unit warps: the products of layer l
        const int g = lane >> 2, q = lane & 3;
        int lseq = 0;    // number of this CTA's stages before the current layer
        int ucount = 0;  // units of this CTA before the current layer
        for (int l = 0; l < a.n_layers; ++l) {
            const ChainLayer ly = tab[l];
            const int K = ly.K, b = l % NB, ph = l / NB;
            const uint8_t *buf = xbase + b * L.buf_bytes;
            const XHeader *hdr = reinterpret_cast<const XHeader *>(buf);
            const int8_t *xq = reinterpret_cast<const int8_t *>(buf + L.off_xq);
            const uint8_t *s_mask = buf + L.off_mask;
            const uint16_t *flaglist = reinterpret_cast<const uint16_t *>(buf + L.off_flaglist);
            const int units = ly.N >> 3, nst = K / ly.seg, segs = ly.seg >> 6;
            const int first = first_unit(ly);
            const int cnt = first < units ? (units - first + grid - 1) / grid : 0;
            const float sw0 = a.per_vec ? 0.0f : __ldg(ly.s_w);
            if (!wait_sleep(&bar_ready[b], (uint32_t)ph & 1u, abort_flag, a.spin)) break;
            const int nflag = hdr->nflag;
            const bool skip = hdr->r > a.cap;  // MUXQ_ERR_CAPACITY: Y of this layer is unspecified; its weights still drain
            for (int i = (warp - ucount) & (kUW - 1); i < cnt; i += kUW) {  // unit number ucount + i goes to warp (ucount + i) mod kUW
                const int u = first + i * grid;
                const int seq0 = lseq + i * nst;
                RingPos pos;
                pos.slot = seq0 % S;
                pos.use = (uint32_t)(seq0 / S);
                // Body accumulators (two: consecutive products on one accumulator wait for each other) and the Aux
                // accumulator over the outlier channels (Aux_q == Body_q[:, O], Eq. 5)
                int accb[4] = {0, 0, 0, 0}, accb2[4] = {0, 0, 0, 0}, acca[4] = {0, 0, 0, 0};
                bool got = true;
                for (int st = 0; st < nst; ++st) {
                    // A barrier phase is told from the one two uses earlier only by its parity, so a warp must not wait
                    // for a stage before the loaders have begun to fill it (by then the slot's previous use has been
                    // consumed and its phase is complete).  With more units per layer than ring slots a warp can get
                    // that far ahead.
                    {
                        uint32_t spins = 0;
                        while (s_begun[pos.slot] <= pos.use && ++spins < a.spin) {
                            __nanosleep(40);
                            if ((spins & 15u) == 15u && *abort_flag) break;
                        }
                        got = __all_sync(0xffffffffu, s_begun[pos.slot] > pos.use);
                        if (!got) *abort_flag = 1u;
                    }
                    got = got && wait_sleep(&bar_full[pos.slot], pos.use & 1u, abort_flag, a.spin);
                    if (!got) break;
                    if (!skip) {
                        // lane (g, q) reads 16 bytes of W_q row 8u + g per 64-byte segment; the matching 16 bytes of the
                        // codes of X come from shared memory.  The K order inside a segment is permuted the same way
                        // for both operands, which a dot product does not notice.  Segments go in batches whose loads
                        // are all issued before the first product (one warp walks a whole unit), with no test of the
                        // outlier flags:
                        const uint8_t *wrow = ring + (size_t)pos.slot * a.slot_bytes + g * ly.seg + q * 16;
                        const int seg0 = st * segs;
                        constexpr int kB = kDotM == 1 ? 4 : 2;
                        auto body = [&](const uint4 &w, const int8_t *xp, int par) {
                            if constexpr (kDotM > 0) {
#pragma unroll
                                for (int m = 0; m < kDotM; ++m) {
                                    const uint4 x = *reinterpret_cast<const uint4 *>(xp + m * L.pitch);
                                    int &acc = par ? accb2[m] : accb[m];
                                    acc = __dp4a((int)w.x, (int)x.x, acc);
                                    acc = __dp4a((int)w.y, (int)x.y, acc);
                                    acc = __dp4a((int)w.z, (int)x.z, acc);
                                    acc = __dp4a((int)w.w, (int)x.w, acc);
                                }
                            } else {
                                const uint4 alo = *reinterpret_cast<const uint4 *>(xp + g * L.pitch);
                                uint4 ahi = make_uint4(0u, 0u, 0u, 0u);
                                if (MT == 16) ahi = *reinterpret_cast<const uint4 *>(xp + (g + 8) * L.pitch);
                                mma_s8(accb, alo.x, ahi.x, alo.y, ahi.y, w.x, w.y);
                                mma_s8(accb2, alo.z, ahi.z, alo.w, ahi.w, w.z, w.w);
                            }
                        };
                        const int8_t *xseg = xq + (size_t)seg0 * 64 + q * 16;
                        int sgi = 0;
                        for (; sgi + kB <= segs; sgi += kB) {
                            uint4 w[kB];
#pragma unroll
                            for (int j = 0; j < kB; ++j) w[j] = *reinterpret_cast<const uint4 *>(wrow + (sgi + j) * 64);
#pragma unroll
                            for (int j = 0; j < kB; ++j) body(w[j], xseg + (sgi + j) * 64, j & 1);
                        }
                        for (; sgi < segs; ++sgi) body(*reinterpret_cast<const uint4 *>(wrow + sgi * 64), xseg + sgi * 64, 0);
                        // ... then the Aux term (Eq. 7) for the few segments of this stage that hold an outlier channel,
                        // from the list the prepare warps made: the same products with X masked to those channels
                        for (int j = 0; j < nflag; ++j) {
                            const int fs = (int)flaglist[j] - seg0;
                            if (fs < 0 || fs >= segs) continue;  // warp-uniform
                            const uint4 w = *reinterpret_cast<const uint4 *>(wrow + fs * 64);
                            const uint4 mk = *reinterpret_cast<const uint4 *>(s_mask + (size_t)(seg0 + fs) * 64 + q * 16);
                            const int8_t *xp = xseg + fs * 64;
                            if constexpr (kDotM > 0) {
#pragma unroll
                                for (int m = 0; m < kDotM; ++m) {
                                    const uint4 x = *reinterpret_cast<const uint4 *>(xp + m * L.pitch);
                                    acca[m] = __dp4a((int)w.x, (int)(x.x & mk.x), acca[m]);
                                    acca[m] = __dp4a((int)w.y, (int)(x.y & mk.y), acca[m]);
                                    acca[m] = __dp4a((int)w.z, (int)(x.z & mk.z), acca[m]);
                                    acca[m] = __dp4a((int)w.w, (int)(x.w & mk.w), acca[m]);
                                }
                            } else {
                                const uint4 alo = *reinterpret_cast<const uint4 *>(xp + g * L.pitch);
                                uint4 ahi = make_uint4(0u, 0u, 0u, 0u);
                                if (MT == 16) ahi = *reinterpret_cast<const uint4 *>(xp + (g + 8) * L.pitch);
                                mma_s8(acca, alo.x & mk.x, ahi.x & mk.x, alo.y & mk.y, ahi.y & mk.y, w.x, w.y);
                                mma_s8(acca, alo.z & mk.z, ahi.z & mk.z, alo.w & mk.w, ahi.w & mk.w, w.z, w.w);
                            }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bar_empty[pos.slot]);  // the stage may be fetched into again
                    pos.advance(1, S);
                }
                if (!got || skip) continue;
                // acc = acc_b + c * acc_a (Eq. 7), dequantization (Eq. 3), store
                auto emit = [&](int m, int n, int acc) {
                    if (m >= M) return;
                    const size_t o = (size_t)m * ly.ldy + n;
                    if (a.out_kind == 2) {
                        reinterpret_cast<int32_t *>(ly.Y)[o] = acc;
                    } else {
                        const float sx = hdr->rowscale[a.per_vec ? m : 0];
                        const float sw = a.per_vec ? __ldg(ly.s_w + n) : sw0;
                        const float y = __fmul_rn(__fmul_rn(sx, sw), __int2float_rn(acc));
                        if (a.out_kind == 1) reinterpret_cast<float *>(ly.Y)[o] = y;
                        else reinterpret_cast<__half *>(ly.Y)[o] = __float2half_rn(y);
                    }
                };
                if constexpr (kDotM > 0) {
                    // the four lanes of a W_q row add up; lane q == 0 of row g holds output channel 8u + g
#pragma unroll
                    for (int m = 0; m < kDotM; ++m) {
                        int v = accb[m] + accb2[m] + a.c * acca[m];
                        v += __shfl_xor_sync(0xffffffffu, v, 1);
                        v += __shfl_xor_sync(0xffffffffu, v, 2);
                        if (q == 0) emit(m, u * 8 + g, v);
                    }
                } else {
                    // this lane holds token rows g and g + 8, output channels 8u + 2q and 8u + 2q + 1
                    emit(g, u * 8 + 2 * q, accb[0] + accb2[0] + a.c * acca[0]);
                    emit(g, u * 8 + 2 * q + 1, accb[1] + accb2[1] + a.c * acca[1]);
                    emit(g + 8, u * 8 + 2 * q, accb[2] + accb2[2] + a.c * acca[2]);
                    emit(g + 8, u * 8 + 2 * q + 1, accb[3] + accb2[3] + a.c * acca[3]);
                }
            }
            ucount += cnt;
            lseq += cnt * nst;
            // this warp is done with the layer's buffer (and has made its stores): one of the kUW arrivals
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_free[b]);
            if (*abort_flag) break;
        }
    }

    // ---------------------------------------------------------------- end
    __syncthreads();
    if (s_abort && t == 0 && a.dev_status) atomicMax(a.dev_status, kStatusTimeout);
}

}  // namespace

bool chain_layer_supported(int M, int K, int N) {
    return M >= 1 && M <= 16 && K >= 64 && K % 64 == 0 && K <= kMaxK && N >= 8 && N % 8 == 0;
}

int chain_slot_bytes(int) { return 10 * 1024; }

int chain_plan(ChainLayer *layers, int n_layers, int grid, int slot_bytes) {
    int kmax = 0, off = 0, waits = 0;
    for (int l = 0; l < n_layers; ++l) {
        ChainLayer &ly = layers[l];
        if (ly.flags & kChainWaitPrev) ly.flags = kChainWaitPrev | (++waits << 1);  // the ordinal of this wait
        int nst = 1;
        while (nst <= ly.K / 64 && !(ly.K % nst == 0 && (ly.K / nst) % 64 == 0 && 8 * (ly.K / nst) <= slot_bytes)) ++nst;
        if (nst > ly.K / 64) return -1;
        ly.seg = ly.K / nst;
        ly.unit_off = off;
        off = (off + (ly.N >> 3)) % grid;
        if (ly.K > kmax) kmax = ly.K;
    }
    return kmax;
}

namespace {

template <int MT, int kDotM>
cudaError_t launch_inst(ChainArgs a, bool cooperative, cudaStream_t s) {
    constexpr int kRows = kDotM > 0 ? kDotM : MT;
    auto kern = k_decode_stream<MT, kDotM>;
    static PerDevice<int> attr_set;
    const int dev = current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    {
        std::lock_guard<std::mutex> lock(device_mutex());
        if (!attr_set.have[dev]) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
            if (e != cudaSuccess) return e;
            attr_set.have[dev] = true;
        }
    }
    // the fp16 rows of X are staged in shared memory one layer ahead when they are few (two copies per group)
    a.stage_x = (kDotM > 0 && a.M <= 2) ? 1 : 0;
    // Small M: several groups of prepare warps, each on a layer of its own (one buffer more than groups); else one
    // group and two buffers when that leaves the ring four stages, one buffer otherwise.
    int slots = 0, fixed = 0;
    int pg = a.n_layers < 2 ? 1 : a.M <= 2 ? 4 : a.M <= 4 ? 2 : 1;
    for (; pg >= 1 && slots < 2; pg >>= 1) {
        for (int nbuf = pg > 1 ? pg + 1 : 2; nbuf >= (pg > 1 ? pg + 1 : 1) && slots < 2; --nbuf) {
            const XLayout L = x_layout(kRows, a.M, a.kmax, a.stage_x != 0, nbuf, pg);
            fixed = a.n_layers * (int)sizeof(ChainLayer) + L.total;
            slots = (kMaxSmem - fixed) / a.slot_bytes;
            if (slots < (nbuf >= 2 ? 4 : 2)) slots = 0;
            a.nbuf = nbuf;
            a.pgroups = pg;
        }
    }
    if (slots > kMaxSlots) slots = kMaxSlots;
    if (slots < 2) return cudaErrorInvalidValue;
    a.lgroups = slots >= kLW ? kLW : 2;
    slots -= slots % a.lgroups;  // a slot keeps its loader warp
    a.slots = slots;
    const size_t smem = (size_t)slots * a.slot_bytes + fixed;
    if (cooperative) {
        void *params[] = {&a};
        return cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(kern), dim3(a.grid), dim3(kThreads), params, smem, s);
    }
    kern<<<a.grid, kThreads, smem, s>>>(a);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode_chain(const ChainArgs &a, bool cooperative, cudaStream_t s) {
    if (a.M == 1) return launch_inst<8, 1>(a, cooperative, s);
    if (a.M <= 4) return launch_inst<8, 4>(a, cooperative, s);
    if (a.M <= 8) return launch_inst<8, 0>(a, cooperative, s);
    return launch_inst<16, 0>(a, cooperative, s);
}

}  // namespace muxq
