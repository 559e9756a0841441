// K3: the uniform INT8 GEMM of Eq. 7 with the Aux correction and the dequantization of Eq. 3 fused
// into one pass:  acc = Body_q.W_q^T + [Aux block].[W_aux block]^T  (int32, TMEM),
//                 Y   = (s_x * s_w) * float(acc).
// The Aux block repeats each Aux column c = 2^exp - 1 times, so the weighted sum of Eq. 7 is a plain
// extension of the K loop by ceil(c*r/32) MMA steps and the accumulator stays a single int32 tile.
//
// sm_100a design: persistent CTAs (one per SM), 128 x BN output tiles, warp-specialised roles:
//   warp 0   TMA producer: 128-byte-swizzled K-major tiles of A (128 x 128 B) and B (BN x 128 B)
//            into a multi-stage shared-memory ring (mbarrier full/empty pairs)
//   warp 1   MMA issuer: tcgen05.mma kind::i8, M=128, N=BN, K=32 per instruction, accumulating in
//            one of two TMEM buffers so the epilogue of tile i overlaps the main loop of tile i+1
//   warps 2-9 epilogue: tcgen05.ld (32 lanes x 32 columns, the next chunk in flight while the current
//            one is converted), int32 -> fp32 -> scale -> fp16/fp32, staged per warp in
//            128-byte-swizzled shared memory (32 rows x 128 B) and written with TMA stores, so
//            global writes are whole 128-byte row segments
// Role dispatch uses a warp index broadcast with a shuffle, which keeps each role's control flow
// and its descriptors / addresses warp-uniform; the producer and the MMA issuer run as whole warps
// with one elected lane issuing (a divergent single-thread loop issues MMAs several times slower).
// Every mbarrier wait is bounded; on expiry the CTA raises MUXQ_ERR_TIMEOUT in the device status
// word, drains its outstanding copies, frees its TMEM and returns.
#include "gemm_common.cuh"

namespace muxq {

namespace {

using namespace gemm;

template <int BN>
struct Cfg {
    static constexpr int kABytes = BM * BK;
    static constexpr int kBBytes = BN * BK;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kTmemCols = 2 * BN;
    static constexpr int kOutBufBytes = 32 * 128;  // one TMA store box: 32 rows x 128 B
    static constexpr int kOutBufs = BN == 256 ? 1 : 2;  // staging buffers per epilogue warp
    static constexpr int kOutBytes = kEpiWarps * kOutBufs * kOutBufBytes;
    static constexpr int kStages = (227 * 1024 - 1024 - kOutBytes - 1024) / kStageBytes;
    static constexpr int kSmemBytes = kStages * kStageBytes + kOutBytes + 1024;  // + alignment slack
    static_assert(kStages >= 3, "operand ring too shallow");
};

template <int BN, int kOut, bool kPerVec, bool kBias>
__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_i8(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_aux,
          const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ CUtensorMap tm_baux,
          const __grid_constant__ CUtensorMap tm_y, const GemmParams p) {
    using C = Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_full[C::kStages], bar_empty[C::kStages], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ uint32_t s_abort;

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);  // warp-uniform by construction
    const int lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - smem_u32(smem_raw));

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tm_a);
        tma_prefetch_desc(&tm_b);
        tma_prefetch_desc(&tm_y);
        if (p.has_aux) {
            tma_prefetch_desc(&tm_aux);
            tma_prefetch_desc(&tm_baux);
        }
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(&bar_full[s], 1);
            mbar_init(&bar_empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bar_acc_full[b], 1);
            mbar_init(&bar_acc_empty[b], kEpiWarps);  // one arrival per epilogue warp
        }
        s_abort = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(&s_tmem_base, C::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, s_tmem_base, 0);
    volatile uint32_t *abort_flag = &s_abort;

    // Aux extent: c*r replicated columns -> at most one extra K block, ceil(c*r/32) MMA steps
    int aux_cols_used = 0;
    if (p.has_aux) aux_cols_used = p.c * min(__ldg(p.n_outliers), p.cap);
    aux_cols_used = __shfl_sync(0xffffffffu, aux_cols_used, 0);
    const int aux_kb = (aux_cols_used + BK - 1) / BK;
    const int total_kb = p.num_kb + aux_kb;
    const int num_tiles = p.tiles_m * p.tiles_n;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (whole warp, one lane issues)
        uint32_t it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
            const int m0 = (tile / p.tiles_n) * BM, n0 = (tile % p.tiles_n) * BN;
            for (int kb = 0; kb < total_kb; ++kb, ++it) {
                const uint32_t s = it % C::kStages, ph = (it / C::kStages) & 1u;
                if (!mbar_wait_warp(&bar_empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                uint8_t *sa = smem_al + s * C::kStageBytes;
                uint8_t *sb = sa + C::kABytes;
                mbar_expect_tx_elect(&bar_full[s], C::kStageBytes);
                if (kb < p.num_kb) {
                    tma_load_2d_elect(sa, &tm_a, &bar_full[s], kb * BK, m0);
                    tma_load_2d_elect(sb, &tm_b, &bar_full[s], kb * BK, n0);
                } else {
                    tma_load_2d_elect(sa, &tm_aux, &bar_full[s], (kb - p.num_kb) * BK, m0);
                    tma_load_2d_elect(sb, &tm_baux, &bar_full[s], (kb - p.num_kb) * BK, n0);
                }
            }
        }
        if (!ok) {
            // drain: wait (bounded) until every copy this warp issued has landed
            const uint32_t first = it > (uint32_t)C::kStages ? it - C::kStages : 0u;
            for (uint32_t j = first; j < it; ++j) {
                const uint32_t s = j % C::kStages, ph = (j / C::kStages) & 1u;
                for (uint32_t i = 0; i < kSpinLimit; ++i)
                    if (__any_sync(0xffffffffu, mbar_try_wait(&bar_full[s], ph))) break;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (whole warp, one lane issues)
        constexpr uint32_t idesc = idesc_i8(BM, BN);
        const uint64_t a_desc0 = smem_desc_sw128(smem_base);
        const uint64_t b_desc0 = smem_desc_sw128(smem_base + C::kABytes);
        const int body_tail_steps = ((p.K - (p.num_kb - 1) * BK) + 31) >> 5;  // valid 32-byte steps of the last body block
        uint32_t it = 0, tile_it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tile_it) {
            const uint32_t buf = tile_it & 1u, aph = (tile_it >> 1) & 1u;
            if (!mbar_wait_warp(&bar_acc_empty[buf], aph ^ 1u, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + buf * BN;
            for (int kb = 0; kb < total_kb; ++kb, ++it) {
                const uint32_t s = it % C::kStages, ph = (it / C::kStages) & 1u;
                if (!mbar_wait_warp(&bar_full[s], ph, abort_flag)) { ok = false; break; }
                tc_fence_after();
                // descriptor start addresses are in 16-byte units: a stage is kStageBytes/16 apart, a 32-byte K step 2
                const uint64_t a_desc = a_desc0 + (uint64_t)(s * (C::kStageBytes >> 4));
                const uint64_t b_desc = b_desc0 + (uint64_t)(s * (C::kStageBytes >> 4));
                int steps = 4;
                if (kb == p.num_kb - 1) steps = body_tail_steps;
                else if (kb >= p.num_kb) steps = (min(BK, aux_cols_used - (kb - p.num_kb) * BK) + 31) >> 5;
                if (steps == 4) {
                    mma_i8_ss_elect(d_tmem, a_desc, b_desc, idesc, kb > 0 ? 1u : 0u);
                    mma_i8_ss_elect(d_tmem, a_desc + 2, b_desc + 2, idesc, 1u);
                    mma_i8_ss_elect(d_tmem, a_desc + 4, b_desc + 4, idesc, 1u);
                    mma_i8_ss_elect(d_tmem, a_desc + 6, b_desc + 6, idesc, 1u);
                } else {
                    for (int k = 0; k < steps; ++k)
                        mma_i8_ss_elect(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                }
                mma_commit_elect(&bar_empty[s]);  // stage reusable once these MMAs have read it
            }
            if (ok) mma_commit_elect(&bar_acc_full[buf]);
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps
        const int quad = warp & 3;           // TMEM lane quadrant this warp may read
        const int chalf = (warp - 2) >> 2;   // which half of the tile's columns this warp converts
        constexpr int kChunks = BN / 2 / 32;                          // 32-column chunks per warp and tile
        constexpr int kChunksPerBox = kOut == kOutF16 ? 2 : 1;        // 128 bytes of output per row and box
        static_assert(kChunks % kChunksPerBox == 0, "a store box must not straddle two warps' columns");
        uint8_t *stage0 = smem_al + C::kStages * C::kStageBytes + (warp - 2) * (C::kOutBufs * C::kOutBufBytes);
        const uint32_t sw_xor = (uint32_t)(lane & 7);
        float sxw = 1.0f, sx = 1.0f;
        if (kOut != kOutI32 && !kPerVec) sxw = __fmul_rn(__ldg(p.s_x), __ldg(p.s_w));
        uint32_t tile_it = 0, n_box = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tile_it) {
            const int m0 = (tile / p.tiles_n) * BM, n0 = (tile % p.tiles_n) * BN;
            const uint32_t buf = tile_it & 1u, aph = (tile_it >> 1) & 1u;
            const int row0 = m0 + quad * 32;
            if (kPerVec && kOut != kOutI32) sx = row0 + lane < p.M ? __ldg(p.s_x + row0 + lane) : 0.0f;
            ok = mbar_wait_warp(&bar_acc_full[buf], aph, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const int col0 = chalf * (BN / 2);
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * BN + col0;
            // Pull this warp's whole share of the accumulator (32 rows x BN/2 columns) into registers at once
            // and hand the TMEM buffer back before converting: the MMA issuer can then start the tile after
            // next while this tile is still being converted and stored.
            uint32_t v[kChunks][32];
#pragma unroll
            for (int ch = 0; ch < kChunks; ++ch) tmem_ld_32x32(taddr + 32 * ch, v[ch]);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_acc_empty[buf]);
#pragma unroll
            for (int ch = 0; ch < kChunks; ++ch) {
                const int piece = ch % kChunksPerBox;  // position of this chunk inside its store box
                uint8_t *stage = stage0 + (n_box % C::kOutBufs) * C::kOutBufBytes;
                if (piece == 0) {
                    // the store that last read this staging buffer must be done reading it
                    if (lane == 0) tma_store_wait_read<C::kOutBufs - 1>();
                    __syncwarp();
                }
                const int gcol = n0 + col0 + 32 * ch;
                convert_chunk<kOut, kPerVec, kBias>(v[ch], reinterpret_cast<uint4 *>(stage + lane * 128),
                                             kOut == kOutF16 ? 4 * piece : 0, sw_xor, sx, sxw, p.s_w + gcol,
                                             p.N - gcol, kBias ? p.bias + gcol : nullptr);
                if (piece == kChunksPerBox - 1) {
                    fence_proxy_async();  // make the generic-proxy writes visible to the TMA engine
                    __syncwarp();
                    if (lane == 0) {
                        // rows >= M and columns >= N are clipped by the copy engine; a box wholly outside is
                        // skipped, but its (empty) group is still committed so the buffer accounting stays exact
                        const int bcol = gcol - 32 * piece;
                        if (row0 < p.M && bcol < p.N) tma_store_2d(&tm_y, stage, bcol, row0);
                        tma_store_commit();
                    }
                    ++n_box;
                }
            }
        }
        // the staging buffers must outlive the copies that read them; the writes themselves complete with the grid
        if (lane == 0) tma_store_wait_read<0>();
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, C::kTmemCols);
    }
    if (threadIdx.x == 0 && s_abort && p.dev_status) atomicMax(p.dev_status, kStatusTimeout);
}

template <int BN, int kOut, bool kPerVec, bool kBias>
cudaError_t launch_gemm_inst(const GemmArgs &a, cudaStream_t s) {
    using C = Cfg<BN>;
    static PerDevice<int> attr_set;  // per instantiation and device
    const int dev = current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    {
        std::lock_guard<std::mutex> lock(device_mutex());
        if (!attr_set.have[dev]) {
            cudaError_t e = cudaFuncSetAttribute(k_gemm_i8<BN, kOut, kPerVec, kBias>,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
            if (e != cudaSuccess) return e;
            attr_set.have[dev] = true;
        }
    }
    const bool has_aux = a.aux_q && a.w_aux && a.n_outliers;
    CUtensorMap tm_a, tm_b, tm_aux, tm_baux, tm_y;
    if (!make_map_out(&tm_y, a.Y, a.M, a.N, a.ldy, a.out_kind)) return cudaErrorInvalidValue;
    if (!make_map_i8(&tm_a, a.body_q, a.M, a.K, a.ld_a, BM)) return cudaErrorInvalidValue;
    if (!make_map_i8(&tm_b, a.w_q, a.N, a.K, a.ldw, BN)) return cudaErrorInvalidValue;
    if (has_aux) {
        if (!make_map_i8(&tm_aux, a.aux_q, a.M, a.aux_cols, a.ld_aux, BM)) return cudaErrorInvalidValue;
        if (!make_map_i8(&tm_baux, a.w_aux, a.N, a.aux_cols, a.ld_waux, BN)) return cudaErrorInvalidValue;
    } else {
        tm_aux = tm_a;
        tm_baux = tm_b;
    }
    GemmParams p;
    p.M = a.M; p.N = a.N; p.K = a.K;
    p.tiles_m = (a.M + BM - 1) / BM;
    p.tiles_n = (a.N + BN - 1) / BN;
    p.num_kb = (a.K + BK - 1) / BK;
    p.has_aux = has_aux ? 1 : 0;
    p.c = a.c; p.cap = a.cap;
    p.n_outliers = a.n_outliers;
    p.s_x = a.s_x;
    p.s_w = a.s_w;
    p.bias = a.out_kind == kOutI32 ? nullptr : a.bias;
    p.dev_status = a.dev_status;
    p.w_stable = 0; p.spin = kSpinLimit; p.skip_kb = -1;
    int grid = p.tiles_m * p.tiles_n;
    if (grid > num_sms()) grid = num_sms();
    k_gemm_i8<BN, kOut, kPerVec, kBias><<<grid, kGemmThreads, C::kSmemBytes, s>>>(tm_a, tm_aux, tm_b, tm_baux, tm_y, p);
    return cudaGetLastError();
}

template <int BN>
cudaError_t launch_gemm_bn(const GemmArgs &a, cudaStream_t s) {
    const bool per_vec = a.s_x_per_row || a.s_w_per_col;  // the two granularities come as a pair
    switch (a.out_kind) {
        case kOutF16:
            if (a.bias) return per_vec ? launch_gemm_inst<BN, kOutF16, true, true>(a, s) : launch_gemm_inst<BN, kOutF16, false, true>(a, s);
            return per_vec ? launch_gemm_inst<BN, kOutF16, true, false>(a, s) : launch_gemm_inst<BN, kOutF16, false, false>(a, s);
        case kOutF32:
            if (a.bias) return per_vec ? launch_gemm_inst<BN, kOutF32, true, true>(a, s) : launch_gemm_inst<BN, kOutF32, false, true>(a, s);
            return per_vec ? launch_gemm_inst<BN, kOutF32, true, false>(a, s) : launch_gemm_inst<BN, kOutF32, false, false>(a, s);
        default: return launch_gemm_inst<BN, kOutI32, false, false>(a, s);
    }
}

}  // namespace

cudaError_t launch_gemm(const GemmArgs &a, cudaStream_t s) {
    // An M128 MMA runs at the full tensor rate for N >= 128.
    // CTA pairs (256-row tiles, a third less operand traffic per SM) unless M is too small to fill them.
    // Measured on B200: with pairs the 256-wide tile is at least as fast as the 128-wide one for every N > 128
    // (the narrower tile needs 1.5x the operand bytes per MMA and becomes load-bound).
    // A 192-wide tile carries 17 % more operand bytes per MMA, but divides some N (768) into fewer idle
    // rounds: take it when its estimated makespan, with a 15 % handicap (measured), still beats the 256-wide one.
    if (a.M > BM && a.N >= 128) {
        int bn = 128;
        if (a.N > 128) {
            const int pairs = num_sms() / 2, tm2 = (a.M + 2 * BM - 1) / (2 * BM);
            const int r256 = (tm2 * ((a.N + 255) / 256) + pairs - 1) / pairs, r192 = (tm2 * ((a.N + 191) / 192) + pairs - 1) / pairs;
            bn = r192 * 192 * 1.15 < r256 * 256.0 ? 192 : 256;
        }
        return launch_gemm_pair(a, bn, s);
    }
    // Single-CTA tiles: 256 halves the operand traffic per MMA; 128 gives more tiles when the 256-wide
    // tiling leaves most of the last wave idle.
    const int sms = num_sms();
    const int tm = (a.M + BM - 1) / BM;
    const int t256 = tm * ((a.N + 255) / 256), t128 = tm * ((a.N + 127) / 128);
    const double w256 = (double)((t256 + sms - 1) / sms) * 2.0, w128 = (double)((t128 + sms - 1) / sms);
    const int bn = (a.N <= 128 || w128 < w256 * 0.9) ? 128 : 256;
    return bn == 128 ? launch_gemm_bn<128>(a, s) : launch_gemm_bn<256>(a, s);
}

}  // namespace muxq
