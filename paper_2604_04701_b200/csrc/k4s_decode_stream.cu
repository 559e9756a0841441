// K4, streaming form: one persistent launch that walks a list of decode-shaped MUXQ layers (M <= 16 token rows
// each; Section III-C, Eq. 1, Eq. 4-5, Eq. 7, Eq. 3 per layer, exactly as the one-layer decode kernel computes
// them).  At these sizes a layer is a stream over its W_q (N*K bytes) and little else, and one launch per layer
// cannot keep HBM busy: a layer moves 1.6-6.6 MB, less than a microsecond of HBM time.  Here the weight stream
// never stops at a layer boundary:
//   producer warp   walks the list of layers and, for every unit of 8 output channels that belongs to this CTA,
//                   fetches the 8 rows of W_q with bulk asynchronous copies into a ring of shared-memory stages
//                   (completion counted in bytes on an mbarrier per stage).  It depends on nothing but the
//                   ring's free slots, so it runs several layers ahead of the arithmetic.
//   consumer warps  per layer: all of them derive the channel maxima, the outlier flags, the scale(s) and the INT8
//                   codes of X into shared memory (redundant per CTA, no grid-wide exchange); then each unit of
//                   the layer is taken by ONE warp, which accumulates the unit's 8 x M outputs over all of K in
//                   registers (4-way byte dot products for M <= 4, mma.sync m16n8k32 above), adds the Aux term of
//                   Eq. 7 for the 64-byte segments that hold an outlier channel, dequantizes and stores.
// Units go to CTAs round-robin with an offset that keeps running from layer to layer, so that the bytes a CTA
// streams even out over a few layers although a single layer rarely divides evenly.
// Layers are independent unless a layer's flags say that its X is written by the layer before it: then the
// consumers pass a bounded grid-wide barrier first (the launch is cooperative); the producer does not.
// All waits are bounded; a wait that runs out raises MUXQ_ERR_TIMEOUT, the copies in flight are awaited and
// every role leaves.  No copy here multicasts.
#include <mutex>

#include "kernels.h"
#include "ptx.cuh"
#include "quant.cuh"

namespace muxq {

namespace {

constexpr int kCW = 16;                 // consumer warps
constexpr int kCT = 32 * kCW;           // consumer threads
constexpr int kThreads = kCT + 32;      // + the producer warp
constexpr int kMaxIter = 2;             // channel groups (8 channels) per consumer thread: K <= 8 * kCT * kMaxIter
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

__device__ __forceinline__ uint4 ld_nc_v4(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void bulk_load(void *smem_dst, const void *gsrc, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void bar_consumers() { asm volatile("bar.sync 1, %0;" ::"n"(kCT) : "memory"); }

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Shared-memory layout behind the ring and the layer table (sized for the widest K of the list).
struct XLayout {
    int pitch;          // bytes per row of X codes; pitch % 128 == 64 keeps the 8-row x 64-byte reads conflict free
    int off_mask;       // [K] 0xFF at outlier channels
    int off_segflag;    // [K/64] segment holds an outlier channel
    int off_grpmask;    // [K/8] per-group flag bits
    int off_xs;         // [MT][K] fp16 copy of X between the two passes (only when it fits), else -1
    int total;
};
__host__ __device__ inline XLayout x_layout(int MT, int K, int budget) {
    XLayout s;
    s.pitch = K + ((64 - (K & 127)) & 127);
    if ((s.pitch & 127) != 64) s.pitch += 64;
    s.off_mask = MT * s.pitch;
    s.off_segflag = s.off_mask + K;
    s.off_grpmask = s.off_segflag + (((K >> 6) + 15) & ~15);
    s.total = (s.off_grpmask + (K >> 3) + 15) & ~15;
    s.off_xs = -1;
    if (s.total + MT * K * 2 <= budget) {
        s.off_xs = s.total;
        s.total += MT * K * 2;
    }
    return s;
}

struct RingPos {
    int slot;
    uint32_t use;
    __device__ __forceinline__ void advance(int n, int S) {  // n < 2 * S
        slot += n;
        while (slot >= S) { slot -= S; ++use; }
    }
};

}  // namespace
