// Issue-bound tcgen05.mma kind::i8 loop: the attainable dense INT8 tensor rate of this GPU at its
// current clocks and power state, used as a roofline denominator next to the nominal figure.
// Every CTA keeps one 128 x 128 B operand A and one N x 128 B operand B resident in shared memory
// (no loads inside the loop) and one thread issues `iters` MMAs of shape M128 x N x K32 into TMEM.
#include "kernels.h"
#include "ptx.cuh"

namespace muxq {

namespace {

template <int BN>
__global__ void __launch_bounds__(128, 1) k_mma_peak(int iters, unsigned long long *cycles_out, int32_t *status) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_done;
    __shared__ uint32_t s_tmem_base, s_abort;
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);  // warp-uniform by construction
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
    for (int i = threadIdx.x; i < (128 + BN) * 128 / 4; i += blockDim.x)
        reinterpret_cast<uint32_t *>(smem_al)[i] = 0x01010101u * (uint32_t)((i * 2654435761u) >> 29);
    if (threadIdx.x == 0) {
        mbar_init(&bar_done, 1);
        s_abort = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(&s_tmem_base, BN < 32 ? 32 : BN);
        tmem_relinquish();
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, s_tmem_base, 0);
    if (warp == 0) {
        constexpr uint32_t idesc = idesc_i8(128, BN);
        const uint32_t a_addr = smem_base, b_addr = smem_base + 128 * 128;
        const long long t0 = clock64();
        for (int i = 0; i < iters; ++i) {
            const int k = i & 3;
            mma_i8_ss_elect(tmem_base, smem_desc_sw128(a_addr + k * 32), smem_desc_sw128(b_addr + k * 32), idesc,
                            i > 0 ? 1u : 0u);
        }
        mma_commit_elect(&bar_done);
        const bool ok = mbar_wait_warp(&bar_done, 0, &s_abort);
        const long long t1 = clock64();
        if ((threadIdx.x & 31) == 0) {
            cycles_out[blockIdx.x] = (unsigned long long)(t1 - t0);
            if (!ok && status) atomicMax(status, 6);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, BN < 32 ? 32 : BN);
    }
}

}  // namespace

cudaError_t launch_mma_peak(int n, int iters, unsigned long long *cycles_out, int32_t *status, int grid,
                            cudaStream_t s) {
    cudaError_t e;
    const int smem = (128 + 256) * 128 + 1024;
    if (n == 256) {
        e = cudaFuncSetAttribute(k_mma_peak<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        k_mma_peak<256><<<grid, 128, smem, s>>>(iters, cycles_out, status);
    } else if (n == 128) {
        e = cudaFuncSetAttribute(k_mma_peak<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        k_mma_peak<128><<<grid, 128, smem, s>>>(iters, cycles_out, status);
    } else if (n == 16) {
        e = cudaFuncSetAttribute(k_mma_peak<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        k_mma_peak<16><<<grid, 128, smem, s>>>(iters, cycles_out, status);
    } else if (n == 64) {
        e = cudaFuncSetAttribute(k_mma_peak<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        k_mma_peak<64><<<grid, 128, smem, s>>>(iters, cycles_out, status);
    } else {
        return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace muxq
