// K3, CTA-pair form: the same INT8 GEMM + Aux + dequantization as k3_gemm.cu, with two CTAs (a cluster
// of 2, two SMs) working on one 256 x BN output tile through tcgen05.mma.cta_group::2.
//
// Why: with one CTA per 128 x 256 tile every SM pulls 48 KB of operands per K block out of L2 and
// through its shared memory, which (together with the epilogue's staging traffic) is what limits the
// single-CTA kernel, not the tensor pipe.  In a pair each CTA loads only ITS 128 rows of A and ITS
// half of B's rows (BN/2); the hardware feeds both tensor cores from both shared memories, so the
// per-SM operand traffic drops by a third for the same MMA work.
//
// Roles per CTA are those of the single-CTA kernel (warp 0 TMA producer, warp 1 MMA issuer, warps 2-9
// epilogue); only the leader CTA (cluster rank 0) issues MMAs.  Synchronisation across the pair:
//   full[s]      lives in the leader; both CTAs' loads complete their bytes on it (the peer's TMA copies
//                name the leader's barrier through its shared::cluster address)
//   empty[s]     one per CTA; the leader's tcgen05.commit arrives on both (commit with a CTA mask)
//   acc_full[b]  one per CTA, same mechanism; each CTA's epilogue drains its own 128 TMEM lanes
//   acc_empty[b] in the leader; the epilogue warps of both CTAs arrive on it (the peer's remotely)
// No TMA copy here multicasts: every CTA fetches its own tiles.  All waits are bounded as in the
// single-CTA kernel; the teardown joins the pair with a cluster barrier before TMEM is released.
#include <cuda_runtime.h>

#include "gemm_common.cuh"

namespace muxq {

namespace {

using namespace gemm;

template <int BN>
struct PairCfg {
    static constexpr int kABytes = BM * BK;          // this CTA's 128 rows of A
    static constexpr int kBBytes = (BN / 2) * BK;    // this CTA's half of B's rows
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kTmemCols = BN > 128 ? 512 : 256;  // two accumulator buffers, a power of two
    static constexpr int kOutBufBytes = 32 * 128;
    static constexpr int kOutBufs = 2;
    static constexpr int kOutBytes = kEpiWarps * kOutBufs * kOutBufBytes;
    static constexpr int kStagesMax = (227 * 1024 - 1024 - kOutBytes - 1024) / kStageBytes;
    static constexpr int kStages = kStagesMax > 8 ? 8 : kStagesMax;
    static constexpr int kSmemBytes = kStages * kStageBytes + kOutBytes + 1024;
    static_assert(kStages >= 4, "operand ring too shallow");
};

template <int BN, int kOut, bool kPerVec, bool kBias>
__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_i8_pair(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_aux,
               const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ CUtensorMap tm_baux,
               const __grid_constant__ CUtensorMap tm_y, const GemmParams p) {
    using C = PairCfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_full[C::kStages], bar_empty[C::kStages], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ uint32_t s_abort;

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);  // warp-uniform by construction
    const int lane = threadIdx.x & 31;
    const uint32_t rank = __shfl_sync(0xffffffffu, cluster_ctarank(), 0);  // 0 = leader; warp-uniform
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
            mbar_init(&bar_full[s], 1);   // the leader's expect_tx arrival; bytes come from both CTAs
            mbar_init(&bar_empty[s], 1);  // the leader's commit
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bar_acc_full[b], 1);
            mbar_init(&bar_acc_empty[b], 2 * kEpiWarps);  // every epilogue warp of both CTAs
        }
        s_abort = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(&s_tmem_base, C::kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // both CTAs' barriers exist before either signals the other's
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, s_tmem_base, 0);
    volatile uint32_t *abort_flag = &s_abort;

    const int num_tiles = p.tiles_m * p.tiles_n;
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    // The weights are constants of the layer: when the caller vouches for that, the producer fetches the B tiles of its
    // first stages before waiting for the predecessor (the preparation of X), whose tail then hides their latency
    // and the first pass through the producer's code.  The A tiles of those stages follow after the wait.
    int pre = 0;
    if (warp == 0 && p.w_stable && pair < num_tiles) {
        pre = min(C::kStages, p.num_kb);
        const int n0 = (pair % p.tiles_n) * BN + (int)rank * (BN / 2);
        for (int kb = 0; kb < pre; ++kb) {
            uint8_t *sb = smem_al + kb * C::kStageBytes + C::kABytes;
            if (rank == 0) mbar_expect_tx_elect(&bar_full[kb], 2 * C::kStageBytes);
            tma_load_2d_pair_elect(sb, &tm_b, map_to_cta(smem_u32(&bar_full[kb]), 0), kb * BK, n0);
        }
    }
    // Launched as a programmatic dependent of the kernel before it in the stream (the activation
    // preparation): the set-up above overlaps that kernel's tail; its results are read only from here on.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // a dependent still waits for this grid to finish

    // r (and with it the number of Aux K blocks) lives in global memory.  It is fetched when a role first reaches the
    // end of a tile's Body blocks, not here: the first operand loads need not wait for that round trip.
    int aux_cols_used = p.has_aux ? -1 : 0, aux_kb = 0;
    auto fetch_aux = [&]() {
        int v = p.c * min(__ldg(p.n_outliers), p.cap);
        aux_cols_used = __shfl_sync(0xffffffffu, v, 0);
        aux_kb = (aux_cols_used + BK - 1) / BK;
    };

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (both CTAs)
        uint32_t it = 0;
        bool ok = true;
        for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
            const int m0 = (tile / p.tiles_n) * (2 * BM) + (int)rank * BM;
            const int n0 = (tile % p.tiles_n) * BN + (int)rank * (BN / 2);
            for (int kb = 0;; ++kb, ++it) {
                if (kb >= p.num_kb) {
                    if (aux_cols_used < 0) fetch_aux();
                    if (kb >= p.num_kb + aux_kb) break;
                }
                const uint32_t s = it % C::kStages, ph = (it / C::kStages) & 1u;
                uint8_t *sa = smem_al + s * C::kStageBytes;
                uint8_t *sb = sa + C::kABytes;
                const uint32_t full_leader = map_to_cta(smem_u32(&bar_full[s]), 0);
                if (it < (uint32_t)pre) {  // stage announced and its B tile already on the way (see above)
                    tma_load_2d_pair_elect(sa, &tm_a, full_leader, kb * BK, m0);
                    continue;
                }
                if (!mbar_wait_warp(&bar_empty[s], ph ^ 1u, abort_flag, p.spin)) { ok = false; break; }
                if (kb == p.skip_kb) continue;  // fault injection (never in normal operation): this stage is never filled
                if (rank == 0) mbar_expect_tx_elect(&bar_full[s], 2 * C::kStageBytes);
                if (kb < p.num_kb) {
                    tma_load_2d_pair_elect(sa, &tm_a, full_leader, kb * BK, m0);
                    tma_load_2d_pair_elect(sb, &tm_b, full_leader, kb * BK, n0);
                } else {
                    tma_load_2d_pair_elect(sa, &tm_aux, full_leader, (kb - p.num_kb) * BK, m0);
                    tma_load_2d_pair_elect(sb, &tm_baux, full_leader, (kb - p.num_kb) * BK, n0);
                }
            }
        }
        if (!ok) {
            // drain: wait (bounded) until the copies issued into this CTA's shared memory have landed.  The
            // leader can watch its full barriers; the peer, whose copies report to the leader, just waits.
            if (rank == 0) {
                const uint32_t first = it > (uint32_t)C::kStages ? it - C::kStages : 0u;
                for (uint32_t j = first; j < it; ++j) {
                    const uint32_t s = j % C::kStages, ph = (j / C::kStages) & 1u;
                    for (uint32_t i = 0; i < p.spin; ++i)
                        if (__any_sync(0xffffffffu, mbar_try_wait(&bar_full[s], ph))) break;
                }
            } else {
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (rank == 0) {
            constexpr uint32_t idesc = idesc_i8(2 * BM, BN);
            const uint64_t a_desc0 = smem_desc_sw128(smem_base);
            const uint64_t b_desc0 = smem_desc_sw128(smem_base + C::kABytes);
            const int body_tail_steps = ((p.K - (p.num_kb - 1) * BK) + 31) >> 5;
            uint32_t it = 0, tile_it = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++tile_it) {
                const uint32_t buf = tile_it & 1u, aph = (tile_it >> 1) & 1u;
                if (!mbar_wait_warp_cluster(&bar_acc_empty[buf], aph ^ 1u, abort_flag, p.spin)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0;; ++kb, ++it) {
                    if (kb >= p.num_kb) {
                        if (aux_cols_used < 0) fetch_aux();
                        if (kb >= p.num_kb + aux_kb) break;
                    }
                    const uint32_t s = it % C::kStages, ph = (it / C::kStages) & 1u;
                    if (!mbar_wait_warp(&bar_full[s], ph, abort_flag, p.spin)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t a_desc = a_desc0 + (uint64_t)(s * (C::kStageBytes >> 4));
                    const uint64_t b_desc = b_desc0 + (uint64_t)(s * (C::kStageBytes >> 4));
                    int steps = 4;
                    if (kb == p.num_kb - 1) steps = body_tail_steps;
                    else if (kb >= p.num_kb) steps = (min(BK, aux_cols_used - (kb - p.num_kb) * BK) + 31) >> 5;
                    if (steps == 4) {
                        mma_i8_ss_pair_elect(d_tmem, a_desc, b_desc, idesc, kb > 0 ? 1u : 0u);
                        mma_i8_ss_pair_elect(d_tmem, a_desc + 2, b_desc + 2, idesc, 1u);
                        mma_i8_ss_pair_elect(d_tmem, a_desc + 4, b_desc + 4, idesc, 1u);
                        mma_i8_ss_pair_elect(d_tmem, a_desc + 6, b_desc + 6, idesc, 1u);
                    } else {
                        for (int k = 0; k < steps; ++k)
                            mma_i8_ss_pair_elect(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc,
                                                 (kb > 0 || k > 0) ? 1u : 0u);
                    }
                    mma_commit_pair_elect(&bar_empty[s]);  // frees stage s in both CTAs
                }
                if (ok) mma_commit_pair_elect(&bar_acc_full[buf]);
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps (both CTAs, own 128 rows)
        const int quad = warp & 3;
        const int chalf = (warp - 2) >> 2;
        // The two warps of a TMEM lane quadrant split the tile's columns in units of 64 (one fp16 store box):
        // the first takes 128 of a 192- or 256-wide tile (64 of a 128-wide one), the second takes the rest.
        constexpr int kCols0 = BN >= 192 ? 128 : BN / 2;
        constexpr int kChunks = kCols0 / 32;              // 32-column chunks of the larger share
        constexpr int kChunksPerBox = kOut == kOutF16 ? 2 : 1;
        static_assert(kChunks % kChunksPerBox == 0 && ((BN - kCols0) / 32) % kChunksPerBox == 0,
                      "a store box must not straddle two warps' columns");
        const int nch = chalf == 0 ? kChunks : (BN - kCols0) / 32;  // warp-uniform
        uint8_t *stage0 = smem_al + C::kStages * C::kStageBytes + (warp - 2) * (C::kOutBufs * C::kOutBufBytes);
        const uint32_t sw_xor = (uint32_t)(lane & 7);
        float sxw = 1.0f, sx = 1.0f;
        if (kOut != kOutI32 && !kPerVec) sxw = __fmul_rn(__ldg(p.s_x), __ldg(p.s_w));
        const uint64_t y_policy = make_policy_evict_first();
        uint32_t tile_it = 0, n_box = 0;
        bool ok = true;
        for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++tile_it) {
            const int m0 = (tile / p.tiles_n) * (2 * BM) + (int)rank * BM, n0 = (tile % p.tiles_n) * BN;
            const uint32_t buf = tile_it & 1u, aph = (tile_it >> 1) & 1u;
            const int row0 = m0 + quad * 32;
            if (kPerVec && kOut != kOutI32) sx = row0 + lane < p.M ? __ldg(p.s_x + row0 + lane) : 0.0f;
            ok = mbar_wait_warp(&bar_acc_full[buf], aph, abort_flag, p.spin);
            if (!ok) break;
            tc_fence_after();
            const int col0 = chalf * kCols0;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * BN + col0;
            // Pull this warp's whole share of the accumulator (32 rows x BN/2 columns) into registers at once
            // and hand the TMEM buffer back before converting: the MMA issuer can then start the tile after
            // next while this tile is still being converted and stored.
            uint32_t v[kChunks][32];
#pragma unroll
            for (int ch = 0; ch < kChunks; ++ch)
                if (ch < nch) tmem_ld_32x32(taddr + 32 * ch, v[ch]);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bar_acc_empty[buf]), 0));
#pragma unroll
            for (int ch = 0; ch < kChunks; ++ch) {
                if (ch >= nch) break;
                const int piece = ch % kChunksPerBox;
                uint8_t *stage = stage0 + (n_box % C::kOutBufs) * C::kOutBufBytes;
                if (piece == 0) {
                    if (lane == 0) tma_store_wait_read<C::kOutBufs - 1>();
                    __syncwarp();
                }
                const int gcol = n0 + col0 + 32 * ch;
                convert_chunk<kOut, kPerVec, kBias>(v[ch], reinterpret_cast<uint4 *>(stage + lane * 128),
                                             kOut == kOutF16 ? 4 * piece : 0, sw_xor, sx, sxw, p.s_w + gcol,
                                             p.N - gcol, kBias ? p.bias + gcol : nullptr);
                if (piece == kChunksPerBox - 1) {
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        const int bcol = gcol - 32 * piece;
                        if (row0 < p.M && bcol < p.N) tma_store_2d_hint(&tm_y, stage, bcol, row0, y_policy);
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
    cluster_sync_all();  // neither CTA releases TMEM (or exits) while the other may still use the pair
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, C::kTmemCols);
    }
    if (threadIdx.x == 0 && s_abort && p.dev_status) atomicMax(p.dev_status, kStatusTimeout);
}

template <int BN, int kOut, bool kPerVec, bool kBias>
cudaError_t launch_pair_inst(const GemmArgs &a, cudaStream_t s) {
    using C = PairCfg<BN>;
    auto kern = k_gemm_i8_pair<BN, kOut, kPerVec, kBias>;
    static PerDevice<int> cache;  // per instantiation and device: clusters of 2 that fit on the device at once
    const int dev = current_device();
    if (dev < 0) return cudaErrorInvalidDevice;
    const int sms = num_sms();
    int max_clusters = 0;
    {
        std::lock_guard<std::mutex> lock(device_mutex());
        if (!cache.have[dev]) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
            if (e != cudaSuccess) return e;
            cudaLaunchConfig_t q{};
            q.gridDim = dim3(2 * sms);
            q.blockDim = dim3(kGemmThreads);
            q.dynamicSmemBytes = C::kSmemBytes;
            cudaLaunchAttribute qa[1];
            qa[0].id = cudaLaunchAttributeClusterDimension;
            qa[0].val.clusterDim.x = 2; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
            q.attrs = qa; q.numAttrs = 1;
            int n = 0;
            e = cudaOccupancyMaxActiveClusters(&n, kern, &q);
            if (e != cudaSuccess) return e;
            if (n < 1) return cudaErrorLaunchOutOfResources;
            cache.v[dev] = n;
            cache.have[dev] = true;
        }
        max_clusters = cache.v[dev];
    }
    const bool has_aux = a.aux_q && a.w_aux && a.n_outliers;
    CUtensorMap tm_a, tm_b, tm_aux, tm_baux, tm_y;
    if (!make_map_out(&tm_y, a.Y, a.M, a.N, a.ldy, a.out_kind)) return cudaErrorInvalidValue;
    if (!make_map_i8(&tm_a, a.body_q, a.M, a.K, a.ld_a, BM)) return cudaErrorInvalidValue;
    if (!make_map_i8(&tm_b, a.w_q, a.N, a.K, a.ldw, BN / 2)) return cudaErrorInvalidValue;
    if (has_aux) {
        if (!make_map_i8(&tm_aux, a.aux_q, a.M, a.aux_cols, a.ld_aux, BM)) return cudaErrorInvalidValue;
        if (!make_map_i8(&tm_baux, a.w_aux, a.N, a.aux_cols, a.ld_waux, BN / 2)) return cudaErrorInvalidValue;
    } else {
        tm_aux = tm_a;
        tm_baux = tm_b;
    }
    GemmParams p;
    p.M = a.M; p.N = a.N; p.K = a.K;
    p.tiles_m = (a.M + 2 * BM - 1) / (2 * BM);
    p.tiles_n = (a.N + BN - 1) / BN;
    p.num_kb = (a.K + BK - 1) / BK;
    p.has_aux = has_aux ? 1 : 0;
    p.c = a.c; p.cap = a.cap;
    p.n_outliers = a.n_outliers;
    p.s_x = a.s_x;
    p.s_w = a.s_w;
    p.bias = a.out_kind == kOutI32 ? nullptr : a.bias;
    p.dev_status = a.dev_status;
    p.w_stable = a.w_stable;
    p.spin = test_hooks().spin_limit ? test_hooks().spin_limit : kSpinLimit;
    p.skip_kb = test_hooks().gemm_skip_kb - 1;
    int clusters = p.tiles_m * p.tiles_n;
    if (clusters > max_clusters) clusters = max_clusters;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(2 * clusters);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, tm_a, tm_aux, tm_b, tm_baux, tm_y, p);
}

template <int BN>
cudaError_t launch_pair_bn(const GemmArgs &a, cudaStream_t s) {
    const bool per_vec = a.s_x_per_row || a.s_w_per_col;
    switch (a.out_kind) {
        case kOutF16:
            if (a.bias) return per_vec ? launch_pair_inst<BN, kOutF16, true, true>(a, s) : launch_pair_inst<BN, kOutF16, false, true>(a, s);
            return per_vec ? launch_pair_inst<BN, kOutF16, true, false>(a, s) : launch_pair_inst<BN, kOutF16, false, false>(a, s);
        case kOutF32:
            if (a.bias) return per_vec ? launch_pair_inst<BN, kOutF32, true, true>(a, s) : launch_pair_inst<BN, kOutF32, false, true>(a, s);
            return per_vec ? launch_pair_inst<BN, kOutF32, true, false>(a, s) : launch_pair_inst<BN, kOutF32, false, false>(a, s);
        default: return launch_pair_inst<BN, kOutI32, false, false>(a, s);
    }
}

}  // namespace

// CTA-pair GEMM; bn = 256, 192 or 128 (tile width).
cudaError_t launch_gemm_pair(const GemmArgs &a, int bn, cudaStream_t s) {
    return bn == 256 ? launch_pair_bn<256>(a, s) : bn == 192 ? launch_pair_bn<192>(a, s) : launch_pair_bn<128>(a, s);
}

}  // namespace muxq
