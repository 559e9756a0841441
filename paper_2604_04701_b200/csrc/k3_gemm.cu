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
//   warps 2-5 epilogue: tcgen05.ld (32 lanes x 32 columns), int32 -> fp32 scale -> fp16/fp32 stores
// Every mbarrier wait is bounded; on expiry the CTA raises MUXQ_ERR_TIMEOUT in the device status
// word, drains its outstanding copies, frees its TMEM and returns.
#include <cuda.h>

#include "kernels.h"
#include "ptx.cuh"

namespace muxq {

namespace {

constexpr int BM = 128;
constexpr int BK = 128;  // bytes of K per stage = one 128-byte swizzle row
constexpr int kGemmThreads = 192;
constexpr int kStatusTimeout = 6;  // MUXQ_ERR_TIMEOUT

template <int BN>
struct Cfg {
    static constexpr int kStages = BN == 256 ? 4 : 6;
    static constexpr int kABytes = BM * BK;
    static constexpr int kBBytes = BN * BK;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kTmemCols = 2 * BN;
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024;  // + alignment slack
};

struct GemmParams {
    int M, N, K;
    int tiles_m, tiles_n;
    int num_kb;    // body K blocks
    int has_aux;   // Aux operands present
    int c, cap;
    const int32_t *n_outliers;
    const float *s_x; int s_x_per_row;
    const float *s_w; int s_w_per_col;
    void *Y; int ldy; int out_kind;
    int32_t *dev_status;
};

template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_i8(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_aux,
          const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ CUtensorMap tm_baux,
          const GemmParams p) {
    using C = Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_full[C::kStages], bar_empty[C::kStages], bar_acc_full[2], bar_acc_empty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ uint32_t s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - smem_u32(smem_raw));

    if (threadIdx.x == 0) {
        tma_prefetch_desc(&tm_a);
        tma_prefetch_desc(&tm_b);
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
            mbar_init(&bar_acc_empty[b], 4);  // one arrival per epilogue warp
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
    const uint32_t tmem_base = s_tmem_base;
    volatile uint32_t *abort_flag = &s_abort;

    // Aux extent: c*r replicated columns -> K blocks and MMA steps of 32
    int aux_cols_used = 0;
    if (p.has_aux && p.n_outliers) aux_cols_used = p.c * min(__ldg(p.n_outliers), p.cap);
    const int aux_kb = (aux_cols_used + BK - 1) / BK;
    const int total_kb = p.num_kb + aux_kb;
    const int num_tiles = p.tiles_m * p.tiles_n;

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------------ TMA producer
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int m0 = (tile / p.tiles_n) * BM, n0 = (tile % p.tiles_n) * BN;
                for (int kb = 0; kb < total_kb; ++kb, ++it) {
                    const uint32_t s = it % C::kStages, ph = (it / C::kStages) & 1u;
                    if (!mbar_wait(&bar_empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t *sa = smem_al + s * C::kStageBytes;
                    uint8_t *sb = sa + C::kABytes;
                    mbar_expect_tx(&bar_full[s], C::kStageBytes);
                    if (kb < p.num_kb) {
                        tma_load_2d(sa, &tm_a, &bar_full[s], kb * BK, m0);
                        tma_load_2d(sb, &tm_b, &bar_full[s], kb * BK, n0);
                    } else {
                        tma_load_2d(sa, &tm_aux, &bar_full[s], (kb - p.num_kb) * BK, m0);
                        tma_load_2d(sb, &tm_baux, &bar_full[s], (kb - p.num_kb) * BK, n0);
                    }
                }
            }
            if (!ok) {
                // drain: wait (bounded) until every copy this thread issued has landed
                const uint32_t first = it > (uint32_t)C::kStages ? it - C::kStages : 0u;
                for (uint32_t j = first; j < it; ++j) {
                    const uint32_t s = j % C::kStages, ph = (j / C::kStages) & 1u;
                    for (uint32_t i = 0; i < kSpinLimit; ++i)
                        if (mbar_try_wait(&bar_full[s], ph)) break;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ------------------------------------------------------------ MMA issuer
            constexpr uint32_t idesc = idesc_i8(BM, BN);
            uint32_t it = 0, tile_it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tile_it) {
                const uint32_t buf = tile_it & 1u, aph = (tile_it >> 1) & 1u;
                if (!mbar_wait(&bar_acc_empty[buf], aph ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < total_kb; ++kb, ++it) {
                    const uint32_t s = it % C::kStages, ph = (it / C::kStages) & 1u;
                    if (!mbar_wait(&bar_full[s], ph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    int k_bytes;  // valid K extent of this block
                    if (kb < p.num_kb) k_bytes = min(BK, p.K - kb * BK);
                    else k_bytes = min(BK, aux_cols_used - (kb - p.num_kb) * BK);
                    const int steps = (k_bytes + 31) >> 5;
                    const uint32_t a_addr = smem_base + s * C::kStageBytes;
                    const uint32_t b_addr = a_addr + C::kABytes;
                    for (int k = 0; k < steps; ++k) {
                        mma_i8_ss(d_tmem, smem_desc_sw128(a_addr + k * 32), smem_desc_sw128(b_addr + k * 32),
                                  idesc, (kb > 0 || k > 0) ? 1u : 0u);
                    }
                    mma_commit(&bar_empty[s]);  // stage reusable once these MMAs have read it
                }
                if (ok) mma_commit(&bar_acc_full[buf]);
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps
        const int quad = warp & 3;  // TMEM lane quadrant this warp may read
        uint32_t tile_it = 0;
        bool ok = true;
        const float sx0 = p.out_kind == 2 ? 1.0f : __ldg(p.s_x);
        const float sw0 = p.out_kind == 2 ? 1.0f : __ldg(p.s_w);
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tile_it) {
            const int m0 = (tile / p.tiles_n) * BM, n0 = (tile % p.tiles_n) * BN;
            const uint32_t buf = tile_it & 1u, aph = (tile_it >> 1) & 1u;
            ok = mbar_wait(&bar_acc_full[buf], aph, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int row = m0 + quad * 32 + lane;
            const bool row_ok = row < p.M;
            float sx = sx0;
            if (p.s_x_per_row && row_ok && p.out_kind != 2) sx = __ldg(p.s_x + row);
#pragma unroll 1
            for (int chunk = 0; chunk < BN / 32; ++chunk) {
                uint32_t v[32];
                __syncwarp();  // tcgen05.ld is warp-collective: reconverge after the guarded stores
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * BN + chunk * 32;
                tmem_ld_32x32(taddr, v);
                tmem_ld_wait();
                const int col0 = n0 + chunk * 32;
                if (!row_ok || col0 >= p.N) continue;
                if (p.out_kind == 2) {
                    int32_t *y = reinterpret_cast<int32_t *>(p.Y) + (size_t)row * p.ldy + col0;
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        if (col0 + g * 4 < p.N)
                            *reinterpret_cast<uint4 *>(y + g * 4) =
                                make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                } else {
                    float f[32];
                    if (p.s_w_per_col) {
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            float4 w4 = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (col0 + g * 4 < p.N) w4 = __ldg(reinterpret_cast<const float4 *>(p.s_w + col0) + g);
                            f[4 * g + 0] = __fmul_rn(__fmul_rn(sx, w4.x), __int2float_rn((int)v[4 * g + 0]));
                            f[4 * g + 1] = __fmul_rn(__fmul_rn(sx, w4.y), __int2float_rn((int)v[4 * g + 1]));
                            f[4 * g + 2] = __fmul_rn(__fmul_rn(sx, w4.z), __int2float_rn((int)v[4 * g + 2]));
                            f[4 * g + 3] = __fmul_rn(__fmul_rn(sx, w4.w), __int2float_rn((int)v[4 * g + 3]));
                        }
                    } else {
                        const float sxw = __fmul_rn(sx, sw0);
#pragma unroll
                        for (int i = 0; i < 32; ++i) f[i] = __fmul_rn(sxw, __int2float_rn((int)v[i]));
                    }
                    if (p.out_kind == 1) {
                        float *y = reinterpret_cast<float *>(p.Y) + (size_t)row * p.ldy + col0;
#pragma unroll
                        for (int g = 0; g < 8; ++g)
                            if (col0 + g * 4 < p.N)
                                *reinterpret_cast<float4 *>(y + g * 4) =
                                    make_float4(f[4 * g], f[4 * g + 1], f[4 * g + 2], f[4 * g + 3]);
                    } else {
                        __half *y = reinterpret_cast<__half *>(p.Y) + (size_t)row * p.ldy + col0;
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            if (col0 + g * 8 < p.N) {
                                __half2 h0 = __floats2half2_rn(f[8 * g + 0], f[8 * g + 1]);
                                __half2 h1 = __floats2half2_rn(f[8 * g + 2], f[8 * g + 3]);
                                __half2 h2 = __floats2half2_rn(f[8 * g + 4], f[8 * g + 5]);
                                __half2 h3 = __floats2half2_rn(f[8 * g + 6], f[8 * g + 7]);
                                uint4 o;
                                o.x = *reinterpret_cast<uint32_t *>(&h0);
                                o.y = *reinterpret_cast<uint32_t *>(&h1);
                                o.z = *reinterpret_cast<uint32_t *>(&h2);
                                o.w = *reinterpret_cast<uint32_t *>(&h3);
                                *reinterpret_cast<uint4 *>(y + g * 8) = o;
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_acc_empty[buf]);
        }
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

// ---------------------------------------------------------------- host side: tensor maps + launch
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// int8 matrix [rows, cols] with pitch ld bytes, K-major; box = 128 bytes x box_rows, 128-byte swizzle.
bool make_map_i8(CUtensorMap *map, const void *ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld};
    cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN>
cudaError_t launch_gemm_bn(const GemmArgs &a, cudaStream_t s) {
    using C = Cfg<BN>;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(k_gemm_i8<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    const bool has_aux = a.aux_q && a.w_aux && a.n_outliers;
    CUtensorMap tm_a, tm_b, tm_aux, tm_baux;
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
    p.s_x = a.s_x; p.s_x_per_row = a.s_x_per_row;
    p.s_w = a.s_w; p.s_w_per_col = a.s_w_per_col;
    p.Y = a.Y; p.ldy = a.ldy; p.out_kind = a.out_kind;
    p.dev_status = a.dev_status;
    int grid = p.tiles_m * p.tiles_n;
    if (grid > num_sms()) grid = num_sms();
    k_gemm_i8<BN><<<grid, kGemmThreads, C::kSmemBytes, s>>>(tm_a, tm_aux, tm_b, tm_baux, p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_gemm(const GemmArgs &a, cudaStream_t s) {
    // Tile width: 256 halves the per-MMA operand traffic; 128 gives more tiles when the 256-wide
    // tiling leaves most of the last wave idle.
    const int sms = num_sms();
    const int tm = (a.M + BM - 1) / BM;
    const int t256 = tm * ((a.N + 255) / 256), t128 = tm * ((a.N + 127) / 128);
    const double w256 = (double)((t256 + sms - 1) / sms) * 2.0, w128 = (double)((t128 + sms - 1) / sms);
    if (a.N <= 128 || w128 < w256 * 0.9) return launch_gemm_bn<128>(a, s);
    return launch_gemm_bn<256>(a, s);
}

}  // namespace muxq
