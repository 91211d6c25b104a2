// Arithmetic of the token-wise symmetric INT8 activation quantizer (Eq. 1 activation side,
// Appendix A.1), shared by the stand-alone quantizer kernel and by the decode kernel that
// quantizes its few tokens itself: both must produce the same bits.
#pragma once

#include "common.cuh"

namespace w4a8 {

__device__ __forceinline__ void scaled8(const uint4 &v, const float *__restrict__ inv_s, int k0,
                                        float (&x)[8])
{
    const __half2 *h2 = reinterpret_cast<const __half2 *>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(h2[i]);
        x[2 * i] = f.x;
        x[2 * i + 1] = f.y;
    }
    if (inv_s) {
        const float4 a = __ldg(reinterpret_cast<const float4 *>(inv_s + k0));
        const float4 b = __ldg(reinterpret_cast<const float4 *>(inv_s + k0 + 4));
        x[0] = __fmul_rn(x[0], a.x); x[1] = __fmul_rn(x[1], a.y);
        x[2] = __fmul_rn(x[2], a.z); x[3] = __fmul_rn(x[3], a.w);
        x[4] = __fmul_rn(x[4], b.x); x[5] = __fmul_rn(x[5], b.y);
        x[6] = __fmul_rn(x[6], b.z); x[7] = __fmul_rn(x[7], b.w);
    }
}

// rint(x * r) clamped to +-127, as the low byte of the result.  The product is rounded to
// binary32 first (as in the reference arithmetic), then adding 1.5 * 2^23 rounds it to an
// integer, half to even, and leaves that integer in the low mantissa bits (two's complement
// in the low byte): two FP32 instructions instead of a float-to-int conversion, which the SM
// issues at an eighth of the FP32 rate and which bounded this kernel.
__device__ __forceinline__ uint32_t round_clamp_bits(float x, float r)
{
    float p = __fmul_rn(x, r);
    p = fminf(fmaxf(p, -127.0f), 127.0f);
    return __float_as_uint(__fadd_rn(p, 12582912.0f));
}

__device__ __forceinline__ uint32_t prmt_b(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

__device__ __forceinline__ uint32_t pack4(const float *x, float r)
{
    const uint32_t a = round_clamp_bits(x[0], r), b = round_clamp_bits(x[1], r);
    const uint32_t c = round_clamp_bits(x[2], r), d = round_clamp_bits(x[3], r);
    // low bytes of a, b, c, d in that order
    return prmt_b(prmt_b(a, b, 0x0040u), prmt_b(c, d, 0x0040u), 0x5410u);
}

__device__ __forceinline__ uint2 quantize8(const float (&x)[8], float r)
{
    uint2 o;
    o.x = pack4(x, r);
    o.y = pack4(x + 4, r);
    return o;
}

}  // namespace w4a8
