// K4, streaming form: one persistent launch that walks a list of decode-shaped MUXQ layers (M <= 16 token rows
// each; Section III-C, Eq. 1, Eq. 4-5, Eq. 7, Eq. 3 per layer, exactly as the one-layer decode kernel computes
// them).  At these sizes a layer is a stream over its W_q (N*K bytes) and little else, and one launch per layer
// cannot keep HBM busy: a layer moves 1.6-6.6 MB, less than a microsecond of HBM time.  Here the weight stream
// never stops at a layer boundary, and the activation work of a layer is done once for the whole grid:
//   loader warps    walk the list of layers and, for every unit of 8 output channels that belongs to this CTA,
//                   fetch the 8 rows of W_q with bulk asynchronous copies (cp.async.bulk, no multicast) into a
//                   ring of shared-memory stages; the copies report their bytes to the stage's mbarrier.  They
//                   depend on nothing but the ring's free slots, so they run several layers ahead of the
//                   arithmetic.  Each loader warp takes every fourth stage on its own: one loop over the stages
//                   (wait for the slot, issue, next) costs a single warp several hundred cycles per stage however
//                   the bytes are moved (measured: 10 KB per 0.3 us, 4.4 TB/s over 148 SMs, with one loop of 128
//                   threads making 16-byte copies; 6.7-7 TB/s with four independent loops), and with one bulk
//                   copy per stage or per row the loop is a few dozen instructions.
//   slice warps     X of a layer is cut into slices of 64 input channels; every slice belongs to one warp of the
//                   grid (round-robin over CTAs, with an offset that keeps running through the list).  Its warp
//                   derives the slice's channel maxima and outlier flags (Section III-C) and merges the maxima of
//                   Body (Eq. 4) into the layer's words in global memory; when all slices of the layer have done so
//                   (a counter), the scale(s) of Eq. 1 are known and the warp writes its slice's INT8 codes and
//                   its outlier mask to the layer's scratch area in global memory and counts itself done.  The
//                   warp whose merge completed the first count writes the layer's header meanwhile (scales, r, the
//                   list of 64-byte segments that hold an outlier channel) and counts that as one more part.
//                   Every CTA used to do all of this for itself, which cost more than the weight stream.
//   fetch warp      per layer, in order: once all parts of the layer are there (one poll looks 32 layers ahead) and one of the
//                   CTA's buffers in shared memory is free, has the copy engine bring header and codes there.
//   unit warps      per layer: each unit is taken by ONE warp, which accumulates the unit's 8 x M outputs over all
//                   of K in registers (4-way byte dot products for M <= 4, mma.sync m16n8k32 above), adds the Aux
//                   term of Eq. 7 for the 64-byte segments that hold an outlier channel, dequantizes and stores.
// Units go to CTAs round-robin with an offset that keeps running from layer to layer, so that the bytes a CTA
// streams even out over a few layers although a single layer rarely divides evenly.
// Layers are independent unless a layer's flags say that its X is written by the layer before it: then the
// slice warps of that layer first wait until every CTA has counted its units of the layer before as stored.
// A warp never waits for a condition that needs one of its own later steps: slices are taken in list order, no
// warp owns two slices of a layer, and the fetch and unit warps only ever wait for earlier layers or for the
// slice warps.  All CTAs are resident (cooperative launch, one CTA per SM).  All waits are bounded; a wait that
// runs out raises MUXQ_ERR_TIMEOUT, tells the other CTAs through a word in global memory, and every role leaves.
#include <mutex>

#include "kernels.h"
#include "ptx.cuh"
#include "quant.cuh"

namespace muxq {

namespace {

constexpr int kUW = 8;                  // unit warps (warps 0..7)
constexpr int kFetch = kUW;             // the fetch warp
constexpr int kSW = kChainSliceWarps;   // slice warps per CTA (the warps behind the fetch warp)
constexpr int kLW = 4;                  // loader warps (warps 16..19)
constexpr int kLoader0 = kUW + 1 + kSW; // index of the first loader warp
constexpr int kThreads = 32 * (kLoader0 + kLW);
constexpr int kMaxK = 8192;             // widest layer: 128 slices
constexpr int kDesc = 16;               // layers whose prepared X can be in shared memory at a time
constexpr int kMaxSlots = 24;
constexpr int kStatusCapacity = 5;      // MUXQ_ERR_CAPACITY
constexpr int kStatusTimeout = 6;       // MUXQ_ERR_TIMEOUT
constexpr int kMaxSmem = 227 * 1024 - 5120;  // dynamic part; the static arrays take about 4.8 KB

__device__ __forceinline__ void mma_s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// `bytes` (a multiple of 16, both addresses 16-byte aligned) global -> shared by the copy engine; the bytes are
// reported to the mbarrier as they land
__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gsrc, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// orders this thread's earlier accesses through ordinary loads and stores (made visible to it by an acquire)
// before its later copies through the copy engine, global memory included
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

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

__device__ __forceinline__ void mbar_arrive_n(uint64_t *bar, uint32_t n) {  // n arrivals at once
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(n) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Bounded wait of a whole converged warp for a counter in global memory to reach `want` (lane 0 polls, with an
// acquire; the warp's later loads are ordered behind it by the shuffle).  A time-out here or anywhere else in the
// grid (the word *g_abort) ends the wait; the first kind also raises both abort flags.
__device__ __forceinline__ bool wait_count(const uint32_t *ctr, uint32_t want, volatile uint32_t *abort_flag,
                                           uint32_t *g_abort, uint32_t limit) {
    int ok = 0;
    if ((threadIdx.x & 31) == 0) {
        bool stopped = false;
        for (uint32_t i = 0; i < limit && !ok && !stopped; ++i) {
            if (ld_acquire_u32(ctr) >= want) ok = 1;
            else {
                __nanosleep(i < 8 ? 100 : 400);
                if ((i & 7u) == 7u) stopped = *abort_flag != 0u || ld_relaxed_u32(g_abort) != 0u;
            }
        }
        if (!ok) {
            *abort_flag = 1u;
            if (!stopped) atomicExch(g_abort, 1u);
        }
    }
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// Per layer, in global memory (zero when the launch starts): the counters and maxima the slice warps share.
struct LayerSync {
    uint32_t merged;      // slices whose maxima and outlier counts are in
    uint32_t coded;       // slices whose codes and mask are written, plus one for the layer's header
    uint32_t r;           // outlier channels found so far
    uint32_t stored;      // CTAs whose units of this layer are stored (counted only when the next layer waits)
    uint32_t bmax[16];    // bit patterns of the row maxima of Body (per tensor: word 0 only)
    uint32_t unused;
    uint32_t pad[11];
};
static_assert(sizeof(LayerSync) == 128, "per-layer words");

// A layer's scratch area in global memory: header block (XHeader, the list of flagged segments, the list of the
// first kChList outlier channels in no particular order), codes [M][K], mask [K] (0xFF at outlier channels),
// segflag [K / 64].
constexpr int kChList = 64;
constexpr int kHeaderBytes = 128, kFlagListBytes = 2 * (kMaxK / 64);
constexpr int kHeadBlock = kHeaderBytes + kFlagListBytes + 2 * kChList;
__host__ __device__ inline size_t scratch_codes_bytes(int M, int K) { return ((size_t)M * K + 127) & ~(size_t)127; }
__host__ __device__ inline size_t scratch_layer_bytes(int M, int K) {
    return (size_t)kHeadBlock + scratch_codes_bytes(M, K) + (size_t)K + (size_t)(((K >> 6) + 127) & ~127);
}

// A layer's prepared X in shared memory.  The outlier mask stays in global memory: only a layer with more than
// kChList outlier channels reads it.  The layers' buffers are cut from one region like from a ring, each as large as
// its own K needs, by the host (chain_geometry): place[l] says where layer l's buffer starts and which earlier layers
// must have been released before it may be filled.
struct XLayout {
    int pitch;          // bytes per row of X codes; pitch % 128 == 64 keeps the 8-row x 64-byte reads conflict free
    int off_flaglist;   // [K/64] u16 behind the 128-byte header: the segments that hold an outlier channel, ascending
    int off_chlist;     // [kChList] u16: outlier channels (all of them when r <= kChList)
    int off_xq;         // [rows][pitch] INT8 codes
    int buf_bytes;
};
__host__ __device__ inline XLayout x_layout(int rows, int K) {
    XLayout s;
    s.pitch = K + ((64 - (K & 127)) & 127);
    if ((s.pitch & 127) != 64) s.pitch += 64;
    s.off_flaglist = kHeaderBytes;
    s.off_chlist = kHeaderBytes + kFlagListBytes;
    s.off_xq = kHeadBlock;
    s.buf_bytes = (s.off_xq + rows * s.pitch + 127) & ~127;
    return s;
}
struct XHeader {        // first bytes of a buffer and of a layer's scratch area
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
    __shared__ uint64_t bar_ready[kDesc], bar_free[kDesc];  // prepared X of layer l (barriers l mod kDesc): filled / no longer read
    __shared__ uint32_t s_abort;
    __shared__ volatile uint32_t s_begun[kMaxSlots];  // uses of a slot the loaders have begun to fill so far
    __shared__ uint32_t s_unitdone[kDesc];            // unit warps that have stored their part of the layer
    __shared__ volatile uint32_t s_fetched[kDesc];    // fetches begun so far for the layers with these barriers
    // per layer, for this CTA: its units, the number of its units before the layer modulo kUW, its stages before the layer
    __shared__ uint16_t s_cnt[kChainMaxLayers];
    __shared__ uint8_t s_uc[kChainMaxLayers];
    __shared__ uint32_t s_lseq[kChainMaxLayers];
    __shared__ uint32_t s_scr[kChainMaxLayers];       // offset of the layer's scratch area
    __shared__ uint32_t s_place[kChainMaxLayers];     // bits 0..15: start of the layer's buffer in 128-byte units; 16..: layers below this one released first

    const int t = threadIdx.x, lane = t & 31;
    const int warp = __shfl_sync(0xffffffffu, t >> 5, 0);  // warp-uniform by construction
    const int S = a.slots, M = a.M;
    // n / S as a multiplication: exact for n * S < 2^32, far beyond any CTA's number of stages (a 32-bit division
    // is some forty instructions, and the warps that need it are single-warp pipelines)
    const uint32_t s_magic = 0xFFFFFFFFu / (uint32_t)S + 1u;
    const int grid = (int)gridDim.x, cta = (int)blockIdx.x;
    uint8_t *ring = smem;
    ChainLayer *tab = reinterpret_cast<ChainLayer *>(smem + (size_t)S * a.slot_bytes);
    uint8_t *xbase = reinterpret_cast<uint8_t *>(tab + a.n_layers);
    volatile uint32_t *abort_flag = &s_abort;
    LayerSync *sync = reinterpret_cast<LayerSync *>(a.sync);
    uint32_t *g_abort = reinterpret_cast<uint32_t *>(sync + a.n_layers);

    // the layer table into shared memory (16-byte pieces), barriers
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(a.layers);
        uint4 *dst = reinterpret_cast<uint4 *>(tab);
        for (int i = t; i < a.n_layers * (int)(sizeof(ChainLayer) / 16); i += kThreads) dst[i] = __ldg(src + i);
        for (int i = t; i < a.n_layers; i += kThreads) s_place[i] = __ldg(a.place + i);
    }
    if (t == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&bar_full[s], 1);    // the loader's arrival that announces the stage's bytes; the copies report them
            mbar_init(&bar_empty[s], 1);   // the one unit warp that took the stage
            s_begun[s] = 0u;
        }
        for (int b = 0; b < kDesc; ++b) {
            mbar_init(&bar_ready[b], 1);   // the fetch warp's arrival that announces the bytes; the copies report them
            mbar_init(&bar_free[b], kUW);  // every unit warp, once per layer
            s_unitdone[b] = 0u;
            s_fetched[b] = 0u;
        }
        s_abort = 0u;
        fence_barrier_init();
    }
    __syncthreads();

    // the units of a layer that belong to this CTA: first, first + grid, ... below N / 8
    auto first_unit = [&](const ChainLayer &ly) {
        int f = cta - (int)ly.unit_off;
        if (f < 0) f += grid;
        return f;
    };
    // How many there are per layer, and the running counts in front of every layer: the warps that have nothing to
    // do in a layer pass it by with two loads.
    for (int l = t; l < a.n_layers; l += kThreads) {
        const ChainLayer &ly = tab[l];
        const int units = ly.N >> 3, first = first_unit(ly);
        const int cnt = first < units ? (units - first + grid - 1) / grid : 0;
        s_cnt[l] = (uint16_t)cnt;
        s_lseq[l] = (uint32_t)(cnt * (int)ly.nst);
        s_scr[l] = (uint32_t)scratch_layer_bytes(kRows, ly.K);
    }
    __syncthreads();
    if (warp == 0) {
        uint32_t carry_u = 0, carry_s = 0, carry_b = 0;
        for (int base = 0; base < a.n_layers; base += 32) {
            const int l = base + lane;
            const bool in = l < a.n_layers;
            const uint32_t c = in ? s_cnt[l] : 0u, st = in ? s_lseq[l] : 0u, sb = in ? s_scr[l] : 0u;
            uint32_t pc = c, ps = st, pb = sb;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t nc = __shfl_up_sync(0xffffffffu, pc, o), nsx = __shfl_up_sync(0xffffffffu, ps, o);
                const uint32_t nb = __shfl_up_sync(0xffffffffu, pb, o);
                if (lane >= o) { pc += nc; ps += nsx; pb += nb; }
            }
            if (in) {
                s_uc[l] = (uint8_t)((carry_u + pc - c) & (kUW - 1));
                s_lseq[l] = carry_s + ps - st;
                s_scr[l] = carry_b + pb - sb;
            }
            carry_u += __shfl_sync(0xffffffffu, pc, 31);
            carry_s += __shfl_sync(0xffffffffu, ps, 31);
            carry_b += __shfl_sync(0xffffffffu, pb, 31);
        }
    }
    __syncthreads();

    if (warp >= kLoader0) {
        // ------------------------------------------------------------ loaders: W_q of every layer, in order.
        // The weights are constants of the layers: nothing here waits for X or a barrier.  Loader warp g fills
        // the stages of this CTA whose running number is g modulo the number of loader warps in use, which
        // divides the number of slots: a slot is always refilled by the warp that filled it before (a warp that
        // met another warp's slot could mistake an older phase of its barrier).
        // A stage is 8 rows of `seg` bytes, stored row after row: one copy when the rows are contiguous in W_q
        // (seg == K == ldw), else one copy per row, issued by 8 lanes.
        const int wl = warp - kLoader0, LG = a.lgroups;
        bool ok = wl < LG;
        for (int l = 0; l < a.n_layers && ok; ++l) {
            const int cnt = (int)s_cnt[l];
            if (cnt == 0) continue;
            const uint32_t lseq = s_lseq[l];  // number of this CTA's stages before the layer
            const ChainLayer ly = tab[l];
            const int seg = (int)ly.seg, nst = (int)ly.nst;
            const int first = first_unit(ly);
            const uint32_t nstage = (uint32_t)(cnt * nst);
            const bool flat = seg == ly.ldw;
            uint32_t j = (uint32_t)(wl - (int)lseq) & (uint32_t)(LG - 1);  // first stage of the layer that is this warp's (LG is 4 or 2)
            int i = (int)j / nst, st = (int)j - i * nst;                                    // its unit and K slice
            for (; j < nstage; j += LG) {
                const uint32_t seq = lseq + j;
                const uint32_t use = __umulhi(seq, s_magic);
                const int slot = (int)(seq - use * (uint32_t)S);
                if (use > 0 && !wait_sleep(&bar_empty[slot], (use - 1u) & 1u, abort_flag, a.spin)) {
                    ok = false;
                    break;
                }
                uint8_t *dst = ring + (size_t)slot * a.slot_bytes;
                const int8_t *src = ly.w_q + (size_t)(first + i * grid) * 8 * ly.ldw + (size_t)st * seg;
                if (lane == 0) {
                    s_begun[slot] = use + 1u;  // the slot's previous use is over: its barrier may be waited on
                    mbar_expect_tx(&bar_full[slot], 8u * (uint32_t)seg);
                }
                __syncwarp();
                if (flat) {
                    if (lane == 0) bulk_load(dst, src, 8u * (uint32_t)seg, &bar_full[slot]);
                } else if (lane < 8) {
                    bulk_load(dst + lane * seg, src + (size_t)lane * ly.ldw, (uint32_t)seg, &bar_full[slot]);
                }
                st += LG;
                while (st >= nst) { st -= nst; ++i; }
            }
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
    } else if (warp == kFetch) {
        // ------------------------------------------------------------ fetch warp: prepared X of layer l into its place
        size_t scr = 0;  // offset of the layer's scratch area
        int ready_upto = 0;  // layers below this one are known to be ready
        int freed = 0;       // layers below this one have been released by the unit warps, in order
        int last_buf = -1;
        uint32_t last_phase = 0;
        for (int l = 0; l < a.n_layers; ++l) {
            const ChainLayer ly = tab[l];
            const int K = ly.K, b = l % kDesc, ph = l / kDesc;
            const XLayout L = x_layout(kRows, K);
            const uint32_t place = s_place[l];
            uint8_t *buf = xbase + (size_t)(place & 0xFFFFu) * 128;
            const uint8_t *g_head = a.scratch + scr;
            const uint8_t *g_codes = g_head + kHeadBlock;
            scr += scratch_layer_bytes(kRows, K);
            // The layers whose space (or whose barriers) this one takes over must have been released, and their copies
            // must have landed (if no unit warp had a unit in such a layer, nobody has waited for them yet).  Layers
            // are waited for in list order, so no barrier is ever more than one phase behind what is asked of it.
            {
                const int upto = max((int)(place >> 16), l - kDesc + 1);  // layers below `upto`
                bool ok = true;
                for (; freed < upto && ok; ++freed)
                    ok = wait_sleep(&bar_free[freed % kDesc], (uint32_t)(freed / kDesc) & 1u, abort_flag, a.spin) &&
                         wait_sleep(&bar_ready[freed % kDesc], (uint32_t)(freed / kDesc) & 1u, abort_flag, a.spin);
                if (!ok) break;
            }
            if (l >= ready_upto) {
                // lane i looks at layer l + i: in a list of independent layers most are ready long before their turn
                bool ok = false, stopped = false;
                for (uint32_t i = 0; i < a.spin && !ok && !stopped; ++i) {
                    const bool rdy = l + lane < a.n_layers &&
                                     ld_acquire_u32(&sync[l + lane].coded) > (uint32_t)(tab[l + lane].K >> 6);  // all slices and the header
                    const uint32_t bal = __ballot_sync(0xffffffffu, rdy);
                    const int n = __ffs((int)~bal) - 1;  // consecutive ready layers from l on (-1: all 32)
                    if (n != 0) {
                        ready_upto = l + (n < 0 ? 32 : n);
                        ok = true;
                    } else {
                        __nanosleep(i < 8 ? 100 : 400);
                        if ((i & 7u) == 7u)
                            stopped = __any_sync(0xffffffffu, *abort_flag != 0u || ld_relaxed_u32(g_abort) != 0u);
                    }
                }
                if (!ok) {
                    if (lane == 0) {
                        *abort_flag = 1u;
                        if (!stopped) atomicExch(g_abort, 1u);
                    }
                    break;
                }
                // headers, codes and masks of the layers found ready, written by other SMs and made visible by the
                // acquire, are ordered before the copy engine reads them
                fence_proxy_async_all();
            }
            if (lane == 0) {
                s_fetched[b] = (uint32_t)ph + 1u;  // the barrier is in this layer's phase: it may be waited on
                mbar_expect_tx(&bar_ready[b], (uint32_t)(kHeadBlock + kRows * K));
            }
            __syncwarp();
            if (lane < kRows) bulk_load(buf + L.off_xq + (size_t)lane * L.pitch, g_codes + (size_t)lane * K, (uint32_t)K, &bar_ready[b]);
            if (lane == 30) bulk_load(buf, g_head, (uint32_t)kHeadBlock, &bar_ready[b]);
            // the unit warps without a unit in this layer pass it by: their arrivals on the buffer's barrier are made here
            // (the barrier is in this layer's phase: the one before was waited for above)
            const int idle = kUW - min((int)s_cnt[l], kUW);
            if (lane == 0 && idle > 0) mbar_arrive_n(&bar_free[b], (uint32_t)idle);
            last_buf = b; last_phase = (uint32_t)ph & 1u;
        }
        // the copies of the last layer fetched have landed before this warp leaves (see the loaders)
        if (last_buf >= 0) {
            bool landed = false;
            for (uint32_t k = 0; k < a.spin && !landed; ++k) landed = mbar_try_wait(&bar_ready[last_buf], last_phase);
        }
    } else if (warp > kFetch) {
        // ------------------------------------------------------------ slice warps
        // Warp number w = (warp index among the slice warps) * grid + cta of the grid's kSW * grid slice warps takes
        // slice s of layer l when (slice_off(l) + s) mod (kSW * grid) == w: consecutive slices go to different CTAs.
        const int NW = kSW * grid, myw = (warp - kFetch - 1) * grid + cta;
        const int rg = lane >> 3, cg = lane & 7;  // this lane: rows rg, rg + 4, rg + 8, rg + 12; channels 8 cg .. 8 cg + 7 of the slice
        const float down = __int_as_float((127 - a.exp_factor) << 23);  // 2^-e
        const float qf = (float)a.qmax;
        size_t scr = 0;
        for (int l = 0; l < a.n_layers; ++l) {
            const ChainLayer ly = tab[l];
            const int K = ly.K, ns = K >> 6;
            uint8_t *g_head = a.scratch + scr;
            uint8_t *g_codes = g_head + kHeadBlock;
            uint8_t *g_mask = g_codes + scratch_codes_bytes(kRows, K);
            uint8_t *g_segflag = g_mask + K;
            scr += scratch_layer_bytes(kRows, K);
            int s = myw - (int)ly.slice_off;
            if (s < 0) s += NW;
            if (s >= ns) continue;
            // X of this layer is Y of the layer before it: every CTA that has units of it must have stored its part
            if ((ly.flags & kChainWaitPrev) &&
                !wait_count(&sync[l - 1].stored, (uint32_t)min(tab[l - 1].N >> 3, grid) + a.extra_arrivals, abort_flag, g_abort, a.spin))
                break;
            const int ch = s * 64 + cg * 8;
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int m = rg + 4 * u;
                v[u] = m < M ? __ldcg(reinterpret_cast<const uint4 *>(ly.X + (size_t)m * ly.ldx + ch)) : make_uint4(0u, 0u, 0u, 0u);
            }
            // channel maxima over the rows (Section III-C): this lane's rows, then the lanes that hold the other rows
            __half2 cm[4];
            cm[0] = cm[1] = cm[2] = cm[3] = __float2half2_rn(0.f);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                cm[0] = __hmax2(cm[0], __habs2(*reinterpret_cast<const __half2 *>(&v[u].x)));
                cm[1] = __hmax2(cm[1], __habs2(*reinterpret_cast<const __half2 *>(&v[u].y)));
                cm[2] = __hmax2(cm[2], __habs2(*reinterpret_cast<const __half2 *>(&v[u].z)));
                cm[3] = __hmax2(cm[3], __habs2(*reinterpret_cast<const __half2 *>(&v[u].w)));
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t w = *reinterpret_cast<uint32_t *>(&cm[i]);
                uint32_t o = __shfl_xor_sync(0xffffffffu, w, 8);
                cm[i] = __hmax2(cm[i], *reinterpret_cast<__half2 *>(&o));
                w = *reinterpret_cast<uint32_t *>(&cm[i]);
                o = __shfl_xor_sync(0xffffffffu, w, 16);
                cm[i] = __hmax2(cm[i], *reinterpret_cast<__half2 *>(&o));
            }
            uint32_t mask = 0;
            float mul[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float c0 = __low2float(cm[i]), c1 = __high2float(cm[i]);
                if (c0 > a.tau) mask |= 1u << (2 * i);  // strict
                if (c1 > a.tau) mask |= 2u << (2 * i);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) mul[i] = (mask >> i) & 1u ? down : 1.0f;
            // maxima of Body (Eq. 4: outlier channels times 2^-e) per row, over the slice's 64 channels
            float rm[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float f[8];
                unpack8(v[u], f);
                float x = 0.0f;
#pragma unroll
                for (int i = 0; i < 8; ++i) x = fmaxf(x, fabsf(f[i] * mul[i]));
                rm[u] = x;
            }
            if (!a.per_vec) rm[0] = fmaxf(fmaxf(rm[0], rm[1]), fmaxf(rm[2], rm[3]));
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (u > 0 && !a.per_vec) break;
                rm[u] = fmaxf(rm[u], __shfl_xor_sync(0xffffffffu, rm[u], 1));
                rm[u] = fmaxf(rm[u], __shfl_xor_sync(0xffffffffu, rm[u], 2));
                rm[u] = fmaxf(rm[u], __shfl_xor_sync(0xffffffffu, rm[u], 4));
            }
            if (a.per_vec) {
                if (cg == 0)
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (rg + 4 * u < M && rm[u] > 0.0f) atomicMax(&sync[l].bmax[rg + 4 * u], __float_as_uint(rm[u]));
            } else {
                rm[0] = fmaxf(rm[0], __shfl_xor_sync(0xffffffffu, rm[0], 8));
                rm[0] = fmaxf(rm[0], __shfl_xor_sync(0xffffffffu, rm[0], 16));
                if (lane == 0 && rm[0] > 0.0f) atomicMax(&sync[l].bmax[0], __float_as_uint(rm[0]));
            }
            {
                // outlier count of the layer; the channels also go to the layer's list, at the places the count
                // hands out (lanes 0..7 hold the slice's eight channel groups)
                const int mine = rg == 0 ? __popc(mask) : 0;
                int pre = mine;
#pragma unroll
                for (int o = 1; o < 8; o <<= 1) {
                    const int n = __shfl_up_sync(0xffffffffu, pre, o);
                    if (cg >= o) pre += n;
                }
                const int total = __shfl_sync(0xffffffffu, pre, 7);
                uint32_t base = 0;
                if (lane == 0 && total > 0) base = atomicAdd(&sync[l].r, (uint32_t)total);
                base = __shfl_sync(0xffffffffu, base, 0);
                if (rg == 0 && mine > 0) {
                    uint16_t *chl = reinterpret_cast<uint16_t *>(g_head + kHeaderBytes + kFlagListBytes);
                    int at = (int)base + pre - mine;
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if ((mask >> i) & 1u) {
                            if (at < kChList) chl[at] = (uint16_t)(ch + i);
                            ++at;
                        }
                }
            }
            {
                const uint32_t any = __ballot_sync(0xffffffffu, mask != 0u);
                if (lane == 0) g_segflag[s] = any ? 1 : 0;
            }
            __syncwarp();
            uint32_t before = 0;
            if (lane == 0) {
                __threadfence();
                before = atomicAdd(&sync[l].merged, 1u);
            }
            before = __shfl_sync(0xffffffffu, before, 0);
            if (before + 1u == (uint32_t)ns) {
                // ---- the last slice of the layer to be merged: everything the header needs is final (maxima, r, the
                // slices' segment flags and channels), so this warp writes it now -- scales, r, flagged 64-byte segments
                // in ascending order, per-layer result -- while the others already quantize, and counts it as one more
                // coded part of the layer
                __threadfence();
                const int rh = (int)__ldcg(&sync[l].r);
                const bool over = rh > a.cap;  // MUXQ_ERR_CAPACITY: no codes were written, Y of this layer is unspecified
                XHeader *hdr = reinterpret_cast<XHeader *>(g_head);
                uint16_t *flaglist = reinterpret_cast<uint16_t *>(g_head + kHeaderBytes);
                float sc0 = 1.0f;
                if (lane < 16) {
                    const float mx = __uint_as_float(__ldcg(&sync[l].bmax[a.per_vec ? lane : 0]));
                    sc0 = mx > 0.0f ? __fdiv_rn(mx, qf) : 1.0f;
                    hdr->rowscale[lane] = sc0;
                }
                uint32_t bits = 0;  // this lane: segments 4 lane .. 4 lane + 3
                if (!over) {
                    const uint32_t w = __ldcg(reinterpret_cast<const uint32_t *>(g_segflag) + lane);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (4 * lane + j < ns && ((w >> (8 * j)) & 0xFFu)) bits |= 1u << j;
                }
                int pre = __popc(bits);  // inclusive prefix count over the lanes
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int n = __shfl_up_sync(0xffffffffu, pre, o);
                    if (lane >= o) pre += n;
                }
                const int nf = __shfl_sync(0xffffffffu, pre, 31);
                int at = pre - __popc(bits);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if ((bits >> j) & 1u) flaglist[at++] = (uint16_t)(4 * lane + j);
                if (lane == 0) {
                    hdr->r = rh;
                    hdr->nflag = nf;
                    if (over && a.dev_status) atomicMax(a.dev_status, kStatusCapacity);
                    if (a.results) {
                        ChainResult rr;
                        rr.n_outliers = rh;
                        rr.status = over ? kStatusCapacity : 0;
                        rr.s_x = sc0;
                        rr.reserved = 0;
                        a.results[l] = rr;
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    __threadfence();
                    atomicAdd(&sync[l].coded, 1u);
                }
            }
            // ---- all slices merged: the scale(s) of Eq. 1 are final; codes of this slice
            if (!wait_count(&sync[l].merged, (uint32_t)ns, abort_flag, g_abort, a.spin)) break;
            const int r = (int)__ldcg(&sync[l].r);
            if (r <= a.cap) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int m = rg + 4 * u;
                    if (m >= M) break;
                    const float mx = __uint_as_float(__ldcg(&sync[l].bmax[a.per_vec ? m : 0]));
                    const float sc = mx > 0.0f ? __fdiv_rn(mx, qf) : 1.0f;
                    float lo, hi;
                    recip_bracket(__frcp_rn(sc), lo, hi);
                    float f[8];
                    unpack8(v[u], f);
#pragma unroll
                    for (int i = 0; i < 8; ++i) f[i] *= mul[i];  // exact
                    uint32_t cb[8];
                    uint2 code;
                    if (quant8_bracket(f, lo, hi, cb)) code = codes_exact(v[u], mask, down, sc, qf);  // rare
                    else code = pack8(cb);
                    *reinterpret_cast<uint2 *>(g_codes + (size_t)m * K + ch) = code;
                }
                if (rg == 0) {
                    uint2 mb;
                    mb.x = ((mask & 1) ? 0xFFu : 0u) | ((mask & 2) ? 0xFF00u : 0u) | ((mask & 4) ? 0xFF0000u : 0u) |
                           ((mask & 8) ? 0xFF000000u : 0u);
                    mb.y = ((mask & 16) ? 0xFFu : 0u) | ((mask & 32) ? 0xFF00u : 0u) | ((mask & 64) ? 0xFF0000u : 0u) |
                           ((mask & 128) ? 0xFF000000u : 0u);
                    *reinterpret_cast<uint2 *>(g_mask + ch) = mb;
                }
            }
            __syncwarp();
            if (lane == 0) {
                __threadfence();
                atomicAdd(&sync[l].coded, 1u);
            }
        }
    } else {
        // ------------------------------------------------------------ unit warps: the products of layer l
        const int g = lane >> 2, q = lane & 3;
        // M <= 4: lane (g, q) reads 16 bytes of W_q row 8u + g per 64-byte segment and the matching 16 bytes of the
        // codes of X.  Segments are taken in pairs, rows with odd g second segment first, so that the eight lanes
        // that shared memory serves together touch all 32 banks (a row is a multiple of 128 bytes long); the K order
        // is permuted the same way for both operands, which a dot product does not notice.
        const int oa = (g & 1) * 64 + q * 16, ob = (1 - (g & 1)) * 64 + q * 16;
        for (int l = 0; l < a.n_layers; ++l) {
            const int cnt = (int)s_cnt[l];
            const int i0 = (warp - (int)s_uc[l]) & (kUW - 1);  // unit number ucount + i of the CTA goes to warp (ucount + i) mod kUW
            if (i0 >= cnt) continue;                             // nothing for this warp in this layer
            const int lseq = (int)s_lseq[l];                     // number of this CTA's stages before the layer
            const ChainLayer ly = tab[l];
            const int K = ly.K, b = l % kDesc, ph = l / kDesc;
            const XLayout L = x_layout(kRows, K);
            const uint8_t *buf = xbase + (size_t)(s_place[l] & 0xFFFFu) * 128;
            const XHeader *hdr = reinterpret_cast<const XHeader *>(buf);
            const int8_t *xq = reinterpret_cast<const int8_t *>(buf + L.off_xq);
            const uint16_t *flaglist = reinterpret_cast<const uint16_t *>(buf + L.off_flaglist);
            const uint16_t *chlist = reinterpret_cast<const uint16_t *>(buf + L.off_chlist);
            const int seg = (int)ly.seg, nst = (int)ly.nst, segs = seg >> 6;
            const int first = first_unit(ly);
            // (a warp that has passed layers by must not take an older phase of the barrier for this one)
            {
                uint32_t spins = 0;
                while (s_fetched[b] <= (uint32_t)ph && ++spins < a.spin) {
                    __nanosleep(100);
                    if ((spins & 15u) == 15u && *abort_flag) break;
                }
                if (!__all_sync(0xffffffffu, s_fetched[b] > (uint32_t)ph)) {
                    *abort_flag = 1u;
                    break;
                }
            }
            if (!wait_sleep(&bar_ready[b], (uint32_t)ph & 1u, abort_flag, a.spin)) break;
            {
                const float ssw0 = a.per_vec ? 0.0f : __fmul_rn(hdr->rowscale[0], __ldg(ly.s_w));  // s_X * s_W (Eq. 3)
                const int r = hdr->r, nflag = hdr->nflag;
                const bool skip = r > a.cap;     // MUXQ_ERR_CAPACITY: Y of this layer is unspecified; its weights still drain
                const bool listed = r <= kChList;  // every outlier channel is in the list
                for (int i = i0; i < cnt; i += kUW) {
                    const int u = first + i * grid;
                    const int seq0 = lseq + i * nst;
                    RingPos pos;
                    pos.use = __umulhi((uint32_t)seq0, s_magic);
                    pos.slot = seq0 - (int)pos.use * S;
                    // Body accumulators (several: consecutive products on one accumulator wait for each other) and the
                    // Aux accumulator over the outlier channels (Aux_q == Body_q[:, O], Eq. 5)
                    constexpr int kAcc = kDotM == 4 ? 2 : 4;
                    int accb[kAcc][4], acca[4] = {0, 0, 0, 0};
#pragma unroll
                    for (int j = 0; j < kAcc; ++j) accb[j][0] = accb[j][1] = accb[j][2] = accb[j][3] = 0;
                    bool got = true;
                    for (int st = 0; st < nst; ++st) {
                        // A barrier phase is told from the one two uses earlier only by its parity, so a warp must not
                        // wait for a stage before the loaders have begun to fill it (by then the slot's previous use has
                        // been consumed and its phase is complete).  With more units per layer than ring slots a warp
                        // can get that far ahead.
                        if (s_begun[pos.slot] <= pos.use) {  // (one load for the whole warp; rarely taken)
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
                            const uint8_t *wst = ring + (size_t)pos.slot * a.slot_bytes;  // the stage: 8 rows of seg bytes
                            const uint8_t *wrow = wst + g * seg;
                            const int k0 = st * seg;
                            const int8_t *xseg = xq + k0;
                            if constexpr (kDotM > 0) {
                                constexpr int kP = kAcc / 2;  // pairs of segments per batch: all loads, then all products
                                int sgi = 0;
                                for (; sgi + 2 * kP <= segs; sgi += 2 * kP) {
                                    uint4 w[2 * kP], x[2 * kP][kDotM];
#pragma unroll
                                    for (int j = 0; j < 2 * kP; ++j) {
                                        const int o = (sgi + (j & ~1)) * 64 + ((j & 1) ? ob : oa);
                                        w[j] = *reinterpret_cast<const uint4 *>(wrow + o);
#pragma unroll
                                        for (int m = 0; m < kDotM; ++m) x[j][m] = *reinterpret_cast<const uint4 *>(xseg + m * L.pitch + o);
                                    }
#pragma unroll
                                    for (int j = 0; j < 2 * kP; ++j)
#pragma unroll
                                        for (int m = 0; m < kDotM; ++m) {
                                            int acc = accb[j][m];
                                            acc = __dp4a((int)w[j].x, (int)x[j][m].x, acc);
                                            acc = __dp4a((int)w[j].y, (int)x[j][m].y, acc);
                                            acc = __dp4a((int)w[j].z, (int)x[j][m].z, acc);
                                            acc = __dp4a((int)w[j].w, (int)x[j][m].w, acc);
                                            accb[j][m] = acc;
                                        }
                                }
                                for (; sgi < segs; ++sgi) {  // what is left, segment by segment in plain order
                                    const int o = sgi * 64 + q * 16;
                                    const uint4 w = *reinterpret_cast<const uint4 *>(wrow + o);
#pragma unroll
                                    for (int m = 0; m < kDotM; ++m) {
                                        const uint4 x = *reinterpret_cast<const uint4 *>(xseg + m * L.pitch + o);
                                        int acc = accb[0][m];
                                        acc = __dp4a((int)w.x, (int)x.x, acc);
                                        acc = __dp4a((int)w.y, (int)x.y, acc);
                                        acc = __dp4a((int)w.z, (int)x.z, acc);
                                        acc = __dp4a((int)w.w, (int)x.w, acc);
                                        accb[0][m] = acc;
                                    }
                                }
                            } else {
                                // mma.sync tiles: lane (g, q) supplies 16 bytes of token rows g and g + 8 and of W_q row
                                // 8u + g per segment (the K order inside a segment permuted alike for both operands)
                                // Four segments at a time, each on an accumulator of its own: all loads, then eight
                                // products in four chains of two.
                                int sgi = 0;
                                for (; sgi + 4 <= segs; sgi += 4) {
                                    uint4 w[4], alo[4], ahi[4];
#pragma unroll
                                    for (int j = 0; j < 4; ++j) {
                                        const int o = (sgi + j) * 64 + q * 16;
                                        w[j] = *reinterpret_cast<const uint4 *>(wrow + o);
                                        alo[j] = *reinterpret_cast<const uint4 *>(xseg + g * L.pitch + o);
                                        ahi[j] = MT == 16 ? *reinterpret_cast<const uint4 *>(xseg + (g + 8) * L.pitch + o) : make_uint4(0u, 0u, 0u, 0u);
                                    }
#pragma unroll
                                    for (int j = 0; j < 4; ++j) mma_s8(accb[j], alo[j].x, ahi[j].x, alo[j].y, ahi[j].y, w[j].x, w[j].y);
#pragma unroll
                                    for (int j = 0; j < 4; ++j) mma_s8(accb[j], alo[j].z, ahi[j].z, alo[j].w, ahi[j].w, w[j].z, w[j].w);
                                }
                                for (; sgi < segs; ++sgi) {
                                    const int o = sgi * 64 + q * 16;
                                    const uint4 w = *reinterpret_cast<const uint4 *>(wrow + o);
                                    const uint4 alo = *reinterpret_cast<const uint4 *>(xseg + g * L.pitch + o);
                                    const uint4 ahi = MT == 16 ? *reinterpret_cast<const uint4 *>(xseg + (g + 8) * L.pitch + o) : make_uint4(0u, 0u, 0u, 0u);
                                    mma_s8(accb[0], alo.x, ahi.x, alo.y, ahi.y, w.x, w.y);
                                    mma_s8(accb[1], alo.z, ahi.z, alo.w, ahi.w, w.z, w.w);
                                }
                            }
                            // ... then the Aux term (Eq. 7) over the outlier channels that fall into this stage
                            if (listed) {
                                // from the channel list: single products W_q[n][k] * X_q[m][k]
                                // (entries in groups of four: the loads of a group do not depend on each other; an entry
                                // outside this stage or past the end of the list reads offset 0 and counts as zero)
                                if constexpr (kDotM > 0) {
                                    // lane (g, q): output channel 8u + g, entries q, q + 4, ... (the four lanes add up below)
                                    for (int o0 = 0; o0 < r; o0 += 16) {
                                        int kk[4], w[4];
#pragma unroll
                                        for (int j = 0; j < 4; ++j) {
                                            const int o = o0 + 4 * j + q;
                                            const int k = (int)chlist[o < kChList ? o : 0] - k0;
                                            const bool in = o < r && (unsigned)k < (unsigned)seg;
                                            kk[j] = in ? k : 0;
                                            w[j] = in ? (int)(int8_t)wrow[kk[j]] : 0;
                                        }
#pragma unroll
                                        for (int j = 0; j < 4; ++j)
#pragma unroll
                                            for (int m = 0; m < kDotM; ++m) acca[m] += w[j] * (int)xseg[m * L.pitch + kk[j]];
                                    }
                                } else {
                                    // lane (g, q): token rows g, g + 8; output channels 8u + 2q, 8u + 2q + 1; every entry
                                    for (int o0 = 0; o0 < r; o0 += 4) {
                                        const uint2 c4 = *reinterpret_cast<const uint2 *>(chlist + o0);
                                        const int ch[4] = {(int)(c4.x & 0xFFFFu), (int)(c4.x >> 16), (int)(c4.y & 0xFFFFu), (int)(c4.y >> 16)};
                                        int kk[4], w0[4], w1[4];
#pragma unroll
                                        for (int j = 0; j < 4; ++j) {
                                            const int k = ch[j] - k0;
                                            const bool in = o0 + j < r && (unsigned)k < (unsigned)seg;
                                            kk[j] = in ? k : 0;
                                            w0[j] = in ? (int)(int8_t)wst[(2 * q) * seg + kk[j]] : 0;
                                            w1[j] = in ? (int)(int8_t)wst[(2 * q + 1) * seg + kk[j]] : 0;
                                        }
#pragma unroll
                                        for (int j = 0; j < 4; ++j) {
                                            const int x0 = (int)xseg[g * L.pitch + kk[j]];
                                            const int x1 = MT == 16 ? (int)xseg[(g + 8) * L.pitch + kk[j]] : 0;
                                            acca[0] += w0[j] * x0;
                                            acca[1] += w1[j] * x0;
                                            acca[2] += w0[j] * x1;
                                            acca[3] += w1[j] * x1;
                                        }
                                    }
                                }
                            } else {
                                // many outlier channels: per flagged 64-byte segment, the same products as for Body with X
                                // masked to the outlier channels
                                // (the mask was written in this launch by other SMs: read through L2; visible by way of the
                                // layer's count of parts and the buffer's barrier)
                                const uint8_t *g_mask = a.scratch + s_scr[l] + kHeadBlock + scratch_codes_bytes(kRows, ly.K);
                                const int seg0 = st * segs;
                                for (int j = 0; j < nflag; ++j) {
                                    const int fs = (int)flaglist[j] - seg0;
                                    if (fs < 0 || fs >= segs) continue;  // warp-uniform
                                    const int o = fs * 64 + q * 16;
                                    const uint4 w = *reinterpret_cast<const uint4 *>(wrow + o);
                                    const uint4 mk = __ldcg(reinterpret_cast<const uint4 *>(g_mask + k0 + o));
                                    if constexpr (kDotM > 0) {
#pragma unroll
                                        for (int m = 0; m < kDotM; ++m) {
                                            const uint4 x = *reinterpret_cast<const uint4 *>(xseg + m * L.pitch + o);
                                            acca[m] = __dp4a((int)w.x, (int)(x.x & mk.x), acca[m]);
                                            acca[m] = __dp4a((int)w.y, (int)(x.y & mk.y), acca[m]);
                                            acca[m] = __dp4a((int)w.z, (int)(x.z & mk.z), acca[m]);
                                            acca[m] = __dp4a((int)w.w, (int)(x.w & mk.w), acca[m]);
                                        }
                                    } else {
                                        const uint4 alo = *reinterpret_cast<const uint4 *>(xseg + g * L.pitch + o);
                                        uint4 ahi = make_uint4(0u, 0u, 0u, 0u);
                                        if (MT == 16) ahi = *reinterpret_cast<const uint4 *>(xseg + (g + 8) * L.pitch + o);
                                        mma_s8(acca, alo.x & mk.x, ahi.x & mk.x, alo.y & mk.y, ahi.y & mk.y, w.x, w.y);
                                        mma_s8(acca, alo.z & mk.z, ahi.z & mk.z, alo.w & mk.w, ahi.w & mk.w, w.z, w.w);
                                    }
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
                            const float ss = a.per_vec ? __fmul_rn(hdr->rowscale[m], __ldg(ly.s_w + n)) : ssw0;
                            float y = __fmul_rn(ss, __int2float_rn(acc));
                            if (ly.bias) y = __fadd_rn(y, __ldg(ly.bias + n));  // the layer's additive term, one fp32 addition
                            if (a.out_kind == 1) reinterpret_cast<float *>(ly.Y)[o] = y;
                            else reinterpret_cast<__half *>(ly.Y)[o] = __float2half_rn(y);
                        }
                    };
                    if constexpr (kDotM > 0) {
                        // The four lanes of a W_q row (output channel 8u + g) add up.  With several token rows the sums
                        // are spread over the four lanes on the way (lane q ends up with row q): three exchanges instead
                        // of eight, and the rows are dequantized and stored side by side.
                        int v[kDotM];
#pragma unroll
                        for (int m = 0; m < kDotM; ++m) {
                            v[m] = a.c * acca[m];
#pragma unroll
                            for (int j = 0; j < kAcc; ++j) v[m] += accb[j][m];
                        }
                        if constexpr (kDotM == 4) {
                            const bool odd = (q & 1) != 0, hi = (q & 2) != 0;
                            const int r0 = __shfl_xor_sync(0xffffffffu, odd ? v[0] : v[1], 1);
                            const int r1 = __shfl_xor_sync(0xffffffffu, odd ? v[2] : v[3], 1);
                            const int k0 = (odd ? v[1] : v[0]) + r0;  // rows 0 (even lanes) / 1 (odd lanes), two lanes' worth
                            const int k1 = (odd ? v[3] : v[2]) + r1;  // rows 2 / 3
                            const int r2 = __shfl_xor_sync(0xffffffffu, hi ? k0 : k1, 2);
                            emit(q, u * 8 + g, (hi ? k1 : k0) + r2);
                        } else if constexpr (kDotM == 2) {
                            const bool odd = (q & 1) != 0;
                            int k0 = (odd ? v[1] : v[0]) + __shfl_xor_sync(0xffffffffu, odd ? v[0] : v[1], 1);
                            k0 += __shfl_xor_sync(0xffffffffu, k0, 2);
                            if (q < 2) emit(q, u * 8 + g, k0);
                        } else {
                            int t0 = v[0] + __shfl_xor_sync(0xffffffffu, v[0], 1);
                            t0 += __shfl_xor_sync(0xffffffffu, t0, 2);
                            if (q == 0) emit(0, u * 8 + g, t0);
                        }
                    } else {
                        // this lane holds token rows g and g + 8, output channels 8u + 2q and 8u + 2q + 1
                        int v[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) v[e] = accb[0][e] + accb[1][e] + accb[2][e] + accb[3][e] + a.c * acca[e];
                        emit(g, u * 8 + 2 * q, v[0]);
                        emit(g, u * 8 + 2 * q + 1, v[1]);
                        emit(g + 8, u * 8 + 2 * q, v[2]);
                        emit(g + 8, u * 8 + 2 * q + 1, v[3]);
                    }
                }
            }
            // this warp is done with the layer's buffer (and has made its stores).  When the next layer reads these
            // stores, the last of the CTA's unit warps with a unit in this layer to get here counts the CTA in (each
            // warp's stores are ordered before its own count by a fence, and all of them before the CTA's by the last
            // warp's).
            __syncwarp();
            if (lane == 0) {
                if (l + 1 < a.n_layers && (tab[l + 1].flags & kChainWaitPrev)) {
                    __threadfence();
                    if (atomicAdd(&s_unitdone[b], 1u) == (uint32_t)(min(cnt, kUW) - 1)) {
                        s_unitdone[b] = 0u;
                        __threadfence();
                        atomicAdd(&sync[l].stored, 1u);
                    }
                }
                mbar_arrive(&bar_free[b]);  // one of the kUW arrivals (the fetch warp has made those of the warps without a unit)
            }
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

size_t chain_sync_bytes(int n_layers) { return (size_t)(n_layers + 1) * sizeof(LayerSync); }

int chain_rows(int M) { return M == 1 ? 1 : M == 2 ? 2 : M <= 4 ? 4 : M <= 8 ? 8 : 16; }

size_t chain_scratch_bytes(const ChainLayer *layers, int n_layers, int M) {
    size_t b = 0;
    for (int l = 0; l < n_layers; ++l) b += scratch_layer_bytes(chain_rows(M), layers[l].K);
    return b;
}

// Shared memory of a CTA: ring stages, the layer table, and a region from which every layer's buffer of prepared X is
// cut in list order, each as large as its own K needs, wrapping around at the end; a buffer may be filled when the
// layers whose buffers it overlaps (all older ones with them: they are released in order) have been released.
// The region gets what holds about six average layers or two of the largest, the ring the rest (two stages per unit
// warp are enough: with one, the stage a warp has just released is refilled with that very warp's next unit and the
// warp sees the whole memory latency on every unit); if that leaves the ring under four stages, the region shrinks
// to two of the largest layers, then to one.
bool chain_geometry(const ChainLayer *layers, int n_layers, int M, int slot_bytes, ChainGeometry *geo, uint32_t *place) {
    const int rows = chain_rows(M);
    const int avail = kMaxSmem - n_layers * (int)sizeof(ChainLayer);
    long long sum = 0;
    int maxbuf = 0;
    for (int l = 0; l < n_layers; ++l) {
        const int b = x_layout(rows, layers[l].K).buf_bytes;
        sum += b;
        if (b > maxbuf) maxbuf = b;
    }
    const int avg = (int)(sum / n_layers);
    int region = 6 * avg > 2 * maxbuf ? 6 * avg : 2 * maxbuf;
    int slots = (avail - region) / slot_bytes;
    if (slots < 4) { region = 2 * maxbuf; slots = (avail - region) / slot_bytes; }
    if (slots < 4) { region = maxbuf; slots = (avail - region) / slot_bytes; }
    if (slots < 2) return false;
    if (slots > 2 * kUW) slots = 2 * kUW;
    geo->lgroups = slots >= kLW ? kLW : 2;
    slots -= slots % geo->lgroups;  // a slot keeps its loader warp
    geo->slots = slots;
    region = (avail - slots * slot_bytes) & ~127;
    if (region > 0xFFFF * 128) region = 0xFFFF * 128;
    geo->xregion = region;
    // the layers' places
    struct Live { int layer, start, end; };
    Live live[kDesc];
    int nlive = 0, head = 0;
    for (int l = 0; l < n_layers; ++l) {
        const int size = x_layout(rows, layers[l].K).buf_bytes;
        if (head + size > region) head = 0;
        const int start = head, end = head + size;
        int upto = 0;  // layers below this one must have been released
        for (;;) {
            bool clash = nlive == kDesc;
            for (int i = 0; i < nlive && !clash; ++i) clash = live[i].start < end && start < live[i].end;
            if (!clash) break;
            upto = live[0].layer + 1;  // the oldest goes, whichever clashed
            for (int i = 1; i < nlive; ++i) live[i - 1] = live[i];
            --nlive;
        }
        live[nlive++] = Live{l, start, end};
        place[l] = (uint32_t)(start / 128) | ((uint32_t)upto << 16);
        head = end;
    }
    return true;
}

int chain_plan(ChainLayer *layers, int n_layers, int grid, int slot_bytes) {
    if (kSW * grid < kMaxK / 64) return -1;  // a warp would own two slices of one layer
    int kmax = 0, off = 0, soff = 0;
    for (int l = 0; l < n_layers; ++l) {
        ChainLayer &ly = layers[l];
        int nst = 1;
        while (nst <= ly.K / 64 && !(ly.K % nst == 0 && (ly.K / nst) % 64 == 0 && 8 * (ly.K / nst) <= slot_bytes)) ++nst;
        if (nst > ly.K / 64) return -1;
        ly.seg = (uint16_t)(ly.K / nst);
        ly.unit_off = (uint16_t)off;
        ly.slice_off = (uint16_t)soff;
        ly.nst = (uint16_t)nst;
        off = (off + (ly.N >> 3)) % grid;
        soff = (soff + (ly.K >> 6)) % (kSW * grid);
        if (ly.K > kmax) kmax = ly.K;
    }
    return kmax;
}

namespace {

template <int MT, int kDotM>
cudaError_t launch_inst(ChainArgs a, cudaStream_t s) {
    // the plan's scratch areas and shared-memory places were laid out for chain_rows(M) rows of codes per layer
    if (chain_rows(a.M) != (kDotM > 0 ? kDotM : MT)) return cudaErrorInvalidValue;
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
    const size_t smem = (size_t)a.slots * a.slot_bytes + (size_t)a.n_layers * sizeof(ChainLayer) + (size_t)a.xregion;
    if (smem > (size_t)kMaxSmem) return cudaErrorInvalidValue;
    void *params[] = {&a};
    return cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(kern), dim3(a.grid), dim3(kThreads), params, smem, s);
}

}  // namespace

cudaError_t launch_decode_chain(const ChainArgs &a, cudaStream_t s) {
    if (a.M == 1) return launch_inst<8, 1>(a, s);
    if (a.M == 2) return launch_inst<8, 2>(a, s);
    if (a.M <= 4) return launch_inst<8, 4>(a, s);
    if (a.M <= 8) return launch_inst<8, 0>(a, s);
    return launch_inst<16, 0>(a, s);
}

}  // namespace muxq
