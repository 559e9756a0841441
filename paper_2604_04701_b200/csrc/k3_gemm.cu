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
//   warps 2-9 epilogue: tcgen05.ld (32 lanes x 32 columns), int32 -> fp32 scale -> fp16/fp32, staged
//            per warp in 128-byte-swizzled shared memory (32 rows x 128 B) and
//            written with TMA stores, so global writes are whole 128-byte row segments
// Every mbarrier wait is bounded; on expiry the CTA raises MUXQ_ERR_TIMEOUT in the device status
// word, drains its outstanding copies, frees its TMEM and returns.
#include <cuda.h>

#include "kernels.h"
#include "ptx.cuh"

namespace muxq {

namespace {

constexpr int BM = 128;
constexpr int BK = 128;  // bytes of K per stage = one 128-byte swizzle row
constexpr int kEpiWarps = 8;                       // two per TMEM lane quadrant, each half of the tile's columns
constexpr int kGemmThreads = 64 + 32 * kEpiWarps;  // TMA warp + MMA warp + epilogue warps
constexpr int kStatusTimeout = 6;  // MUXQ_ERR_TIMEOUT

template <int BN>
struct Cfg {
    static constexpr int kStages = BN == 256 ? 4 : 6;
    static constexpr int kABytes = BM * BK;
    static constexpr int kBBytes = BN * BK;
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kTmemCols = 2 * BN;
    static constexpr int kOutStageBytes = 32 * 128;                  // 32 rows x 128 B per epilogue warp
    static constexpr int kOutBytes = kEpiWarps * kOutStageBytes;
    static constexpr int kSmemBytes = kStages * kStageBytes + kOutBytes + 1024;  // + alignment slack
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
    int dbg;
    long long *tl;  // debug timeline (CTA 0): [0..255] producer, [256..511] mma, [512..767] epilogue warp 2
};

// int32 -> fp32, round to nearest even, exact for every int32, without the (slow) conversion unit:
// a = hi * 65536 + lo with lo in [0, 65535]; both halves become floats by the "magic constant" bit
// trick (2^23 + lo, 1.5 * 2^23 + hi, minus the constant) and one fused multiply-add rounds once.
__device__ __forceinline__ float i32_to_f32_rn(int a) {
    const float flo = __uint_as_float(0x4B000000u | ((uint32_t)a & 0xFFFFu)) - 8388608.0f;
    const float fhi = __int_as_float(0x4B400000 + (a >> 16)) - 12582912.0f;
    return fmaf(fhi, 65536.0f, flo);
}

template <int BN>
__global__ void __launch_bounds__(kGemmThreads, 1)
k_gemm_i8(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_aux,
          const __grid_constant__ CUtensorMap tm_b, const __grid_constant__ CUtensorMap tm_baux,
          const __grid_constant__ CUtensorMap tm_y, const GemmParams p) {
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
                    if (p.tl && blockIdx.x == 0 && it < 256) p.tl[it] = clock64();
                    uint8_t *sa = smem_al + s * C::kStageBytes;
                    uint8_t *sb = sa + C::kABytes;
                    if (p.dbg & 2) { mbar_arrive(&bar_full[s]); continue; }
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
                    if (p.tl && blockIdx.x == 0 && it < 256) p.tl[256 + it] = clock64();
                    tc_fence_after();
                    int k_bytes;  // valid K extent of this block
                    if (kb < p.num_kb) k_bytes = min(BK, p.K - kb * BK);
                    else k_bytes = min(BK, aux_cols_used - (kb - p.num_kb) * BK);
                    const int steps = (k_bytes + 31) >> 5;
                    const uint32_t a_addr = smem_base + s * C::kStageBytes;
                    const uint32_t b_addr = a_addr + C::kABytes;
                    for (int k = 0; k < ((p.dbg & 4) ? 0 : steps); ++k) {
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
        uint32_t tile_it = 0, n_store = 0;
        bool ok = true;
        const bool raw = p.out_kind == 2;
        const int cmode = (p.dbg >> 9) & 3;
        const float sx0 = raw ? 1.0f : __ldg(p.s_x);
        const float sw0 = raw ? 1.0f : __ldg(p.s_w);
        const int cols_per_chunk = p.out_kind == 0 ? 64 : 32;  // 128 bytes of output per row
        const int chalf = (warp - 2) >> 2;  // which half of the tile's columns this warp converts
        uint8_t *stage = smem_al + C::kStages * C::kStageBytes + (warp - 2) * C::kOutStageBytes;
        const uint32_t sw_xor = (uint32_t)(lane & 7);
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tile_it) {
            const int m0 = (tile / p.tiles_n) * BM, n0 = (tile % p.tiles_n) * BN;
            const uint32_t buf = tile_it & 1u, aph = (tile_it >> 1) & 1u;
            ok = mbar_wait(&bar_acc_full[buf], aph, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (p.tl && blockIdx.x == 0 && warp == 2 && lane == 0 && tile_it < 100) p.tl[512 + 2 * tile_it] = clock64();
            tc_fence_after();
            const int row0 = m0 + quad * 32;
            const int row = row0 + lane;
            float sx = sx0;
            if (p.s_x_per_row && row < p.M && !raw) sx = __ldg(p.s_x + row);
            const float sxw0 = __fmul_rn(sx, sw0);
#pragma unroll 1
            for (int col = chalf * (BN / 2); col < (chalf + 1) * (BN / 2); col += cols_per_chunk) {
                const int gcol = n0 + col;
                if (p.dbg & 128) { ++n_store; continue; }
                uint4 *srow = reinterpret_cast<uint4 *>(stage + lane * 128);
                const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * BN + col;
                if (p.out_kind == 0) {
                    uint32_t v0[32], v1[32];
                    tmem_ld_32x32(taddr, v0);
                    tmem_ld_32x32(taddr + 32, v1);
                    tmem_ld_wait();
                    // the TMA store that last read the staging buffer must be done with it
                    if (lane == 0) tma_store_wait_read<0>();
                    __syncwarp();
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        float f[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int idx = g * 8 + i;
                            const int a = (int)(idx < 32 ? v0[idx & 31] : v1[idx & 31]);
                            float sc = sxw0;
                            if (p.s_w_per_col) sc = __fmul_rn(sx, gcol + idx < p.N ? __ldg(p.s_w + gcol + idx) : 0.0f);
                            f[i] = __fmul_rn(sc, (cmode == 1 || (cmode == 2 && (i & 3) == 0)) ? __int2float_rn(a) : i32_to_f32_rn(a));
                        }
                        __half2 h0 = __floats2half2_rn(f[0], f[1]), h1 = __floats2half2_rn(f[2], f[3]);
                        __half2 h2 = __floats2half2_rn(f[4], f[5]), h3 = __floats2half2_rn(f[6], f[7]);
                        uint4 o;
                        o.x = *reinterpret_cast<uint32_t *>(&h0); o.y = *reinterpret_cast<uint32_t *>(&h1);
                        o.z = *reinterpret_cast<uint32_t *>(&h2); o.w = *reinterpret_cast<uint32_t *>(&h3);
                        srow[g ^ sw_xor] = o;
                    }
                } else {
                    uint32_t v[32];
                    tmem_ld_32x32(taddr, v);
                    tmem_ld_wait();
                    if (lane == 0) tma_store_wait_read<0>();
                    __syncwarp();
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        uint4 o;
                        if (raw) {
                            o = make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                        } else {
                            float f[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int idx = g * 4 + i;
                                float sc = sxw0;
                                if (p.s_w_per_col)
                                    sc = __fmul_rn(sx, gcol + idx < p.N ? __ldg(p.s_w + gcol + idx) : 0.0f);
                                f[i] = __fmul_rn(sc, (cmode == 1 || (cmode == 2 && (i & 3) == 0)) ? __int2float_rn((int)v[idx]) : i32_to_f32_rn((int)v[idx]));
                            }
                            o = make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                                           __float_as_uint(f[3]));
                        }
                        srow[g ^ sw_xor] = o;
                    }
                }
                if (!(p.dbg & 64)) fence_proxy_async();  // make the generic-proxy writes visible to the TMA engine
                __syncwarp();
                if (lane == 0) {
                    // rows >= M and columns >= N are clipped by the copy engine; a chunk wholly outside is
                    // skipped, but its (empty) group is still committed so the buffer accounting stays exact
                    if (row0 < p.M && gcol < p.N && !(p.dbg & 1)) tma_store_2d(&tm_y, stage, gcol, row0);
                    tma_store_commit();
                }
                ++n_store;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_acc_empty[buf]);
            if (p.tl && blockIdx.x == 0 && warp == 2 && lane == 0 && tile_it < 100) p.tl[513 + 2 * tile_it] = clock64();
        }
        if (lane == 0) tma_store_wait_all<0>();
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

// output matrix [M, N] of 2- or 4-byte elements, pitch ldy elements; box = 128 bytes x 32 rows
bool make_map_out(CUtensorMap *map, void *ptr, uint64_t rows, uint64_t cols, uint64_t ldy, int out_kind) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const uint64_t esz = out_kind == 0 ? 2 : 4;
    const CUtensorMapDataType dt = out_kind == 0   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                   : out_kind == 1 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                                   : CU_TENSOR_MAP_DATA_TYPE_INT32;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ldy * esz};
    cuuint32_t box[2] = {(cuuint32_t)(128 / esz), 32};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, dt, 2, ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int g_dbg = 0;
long long *g_tl = nullptr;

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
    p.s_x = a.s_x; p.s_x_per_row = a.s_x_per_row;
    p.s_w = a.s_w; p.s_w_per_col = a.s_w_per_col;
    p.Y = a.Y; p.ldy = a.ldy; p.out_kind = a.out_kind;
    p.dev_status = a.dev_status;
    p.dbg = g_dbg;
    p.tl = g_tl;
    int grid = p.tiles_m * p.tiles_n;
    if (grid > num_sms()) grid = num_sms();
    k_gemm_i8<BN><<<grid, kGemmThreads, C::kSmemBytes, s>>>(tm_a, tm_aux, tm_b, tm_baux, tm_y, p);
    return cudaGetLastError();
}

}  // namespace

void set_gemm_dbg(int v) { g_dbg = v; }
void set_gemm_tl(long long *p) { g_tl = p; }

cudaError_t launch_gemm(const GemmArgs &a, cudaStream_t s) {
    if (g_dbg & 8) return launch_gemm_bn<256>(a, s);
    if (g_dbg & 16) return launch_gemm_bn<128>(a, s);
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
