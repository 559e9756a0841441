// Device helpers shared by the activation-quantization kernels: Eq. 1 codes equal to
// round_half_even(v / s) with a true fp32 division (bit for bit), and fp16 unpacking.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace muxq {

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Eq. 1: code = clamp(round_half_even(v / s), -q, q) with a true fp32 division.
__device__ __forceinline__ int quant_exact(float v, float s, float qf) {
    float t = rintf(__fdiv_rn(v, s));
    t = fminf(fmaxf(t, -qf), qf);
    return __float2int_rn(t);
}

__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8]) {
    const __half2 *h = reinterpret_cast<const __half2 *>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 p = __half22float2(h[i]);
        f[2 * i] = p.x;
        f[2 * i + 1] = p.y;
    }
}

// 8 values (already multiplied by their channel factors) -> 8 codes packed in a uint2.
//
// Fast path: p = v * (1/s), taken exactly inside a fused multiply-add, differs from the correctly
// rounded quotient v / s by less than 1.6e-5 for |v/s| <= 128, so whenever p is farther than 1e-4
// from every half-integer both round to the same integer.  fma(v, 1/s, 1.5 * 2^23) rounds p to that
// integer (round half to even) and leaves its two's-complement low byte in the low byte of the
// float's bit pattern, which a byte permute packs directly; a second fma gives p minus that integer.
// If any of the 8 values is too close to a tie, or exceeds the code range (possible only when the
// scale was not derived from these values), all 8 take the exact division.
__device__ __forceinline__ uint2 quant8(const float (&f)[8], float s, float inv_s, float qf) {
    const float magic = 12582912.0f;  // 1.5 * 2^23
    uint32_t b[8];
    float dmax = 0.0f, amax = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float tm = fmaf(f[i], inv_s, magic);
        const float n = tm - magic;
        dmax = fmaxf(dmax, fabsf(fmaf(f[i], inv_s, -n)));
        amax = fmaxf(amax, fabsf(n));
        b[i] = __float_as_uint(tm);
    }
    if (dmax > 0.4999f || amax > qf) {
#pragma unroll
        for (int i = 0; i < 8; ++i) b[i] = (uint32_t)quant_exact(f[i], s, qf);
    }
    const uint32_t p01 = __byte_perm(b[0], b[1], 0x0040), p23 = __byte_perm(b[2], b[3], 0x0040);
    const uint32_t p45 = __byte_perm(b[4], b[5], 0x0040), p67 = __byte_perm(b[6], b[7], 0x0040);
    return make_uint2(__byte_perm(p01, p23, 0x5410), __byte_perm(p45, p67, 0x5410));
}

// Bracket form of the fast path, for a scale s that was derived from the values themselves (no code can leave
// [-q, q]).  With inv = RN(1/s), the correctly rounded quotient RN(v/s) differs from the real product v * inv
// by a relative 2^-23 (1 + 2^-23) at most, so it lies between v * lo and v * hi for lo / hi three units in the
// last place below / above inv.  fma(v, lo, 1.5 * 2^23) and fma(v, hi, 1.5 * 2^23) round those two real products
// to integers (half to even) exactly once each; rounding to an integer is monotone, so when both give the same
// integer, round_half_even(RN(v/s)) is that integer too, and its two's-complement low byte sits in the low byte
// of the float's bit pattern.  Power-of-two channel factors folded into lo / hi keep all of this exact.
// Returns nonzero when some value sits too close to a tie for the bracket to decide; the caller then takes
// the exact division for the chunk.  Three instructions per value (two fma, one logic op).
__device__ __forceinline__ void recip_bracket(float inv_s, float &lo, float &hi) {
    lo = __uint_as_float(__float_as_uint(inv_s) - 3u);  // inv_s is a positive normal number
    hi = __uint_as_float(__float_as_uint(inv_s) + 3u);
}

__device__ __forceinline__ uint32_t quant8_bracket(const float (&f)[8], const float (&lo)[8], const float (&hi)[8],
                                                   uint32_t (&b)[8]) {
    const float magic = 12582912.0f;  // 1.5 * 2^23
    uint32_t diff = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        b[i] = __float_as_uint(fmaf(f[i], hi[i], magic));
        diff |= b[i] ^ __float_as_uint(fmaf(f[i], lo[i], magic));
    }
    return diff;
}

__device__ __forceinline__ uint32_t quant8_bracket(const float (&f)[8], float lo, float hi, uint32_t (&b)[8]) {
    const float magic = 12582912.0f;
    uint32_t diff = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        b[i] = __float_as_uint(fmaf(f[i], hi, magic));
        diff |= b[i] ^ __float_as_uint(fmaf(f[i], lo, magic));
    }
    return diff;
}

// low bytes of 8 words -> 8 codes in a uint2
__device__ __forceinline__ uint2 pack8(const uint32_t (&b)[8]) {
    const uint32_t p01 = __byte_perm(b[0], b[1], 0x0040), p23 = __byte_perm(b[2], b[3], 0x0040);
    const uint32_t p45 = __byte_perm(b[4], b[5], 0x0040), p67 = __byte_perm(b[6], b[7], 0x0040);
    return make_uint2(__byte_perm(p01, p23, 0x5410), __byte_perm(p45, p67, 0x5410));
}

// The exact form of Eq. 1 for one 8-channel chunk (mask: its outlier channels).  Kept out of line: it runs for
// about one chunk in a thousand, and inlined at every use it costs the quantization loops their registers.
static __device__ __noinline__ uint2 codes_exact(uint4 v, uint32_t mask, float down, float s, float qf) {
    float f[8];
    unpack8(v, f);
    uint32_t code[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) code[i] = (uint32_t)quant_exact((mask >> i) & 1u ? f[i] * down : f[i], s, qf);
    return pack8(code);
}

}  // namespace muxq
