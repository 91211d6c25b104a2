// Token-wise INT8 activation quantizer: Q(diag(s)^-1 X) of Eq. 1 (Appendix A.1,
// "token-wise quantization for activations"), symmetric absmax variant.
// A token stays in registers between the absmax pass and the rounding pass, so HBM sees 2
// bytes read and 1 byte written per element.  For K <= 16384 the streaming kernels run: tokens
// walk through resident CTAs whose threads keep their reciprocal scales in registers.  Longer
// tokens take the one-token-per-CTA kernels.
#include "common.cuh"
#include "quant_math.cuh"

namespace w4a8 {

namespace {

constexpr int kActThreads = 256;

__device__ __forceinline__ float block_max(float v, float *smem)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if ((threadIdx.x & 31) == 0) smem[threadIdx.x >> 5] = v;
    __syncthreads();
    float m = smem[0];
#pragma unroll
    for (int w = 1; w < kActThreads / 32; ++w) m = fmaxf(m, smem[w]);
    return m;
}

// NV = 16-byte vectors per thread held in registers (K <= 2048 * NV); NV == 0 re-reads
// the token from global memory (L2) in the second pass, for any K.
template <int NV>
__global__ void __launch_bounds__(kActThreads)
act_quant_kernel(const __half *__restrict__ X, const float *__restrict__ inv_s, int M, int K,
                 int8_t *__restrict__ Xq, float *__restrict__ tok_scale)
{
    __shared__ float red[kActThreads / 32];
    allow_dependents();
    dependent_wait();                      // X may be the output of the kernel before
    const int m = blockIdx.x;
    const int tid = threadIdx.x;
    const int nvec = K >> 3;
    const uint4 *row = reinterpret_cast<const uint4 *>(X + (size_t)m * K);
    uint2 *out = reinterpret_cast<uint2 *>(Xq + (size_t)m * K);
    constexpr int NR = NV > 0 ? NV : 1;
    uint4 v[NR];
    float amax = 0.0f;
    if (NV > 0) {
#pragma unroll
        for (int i = 0; i < NR; ++i) {
            const int idx = tid + i * kActThreads;
            v[i] = make_uint4(0u, 0u, 0u, 0u);
            if (idx < nvec) v[i] = __ldcs(row + idx);
        }
#pragma unroll
        for (int i = 0; i < NR; ++i) {
            const int idx = tid + i * kActThreads;
            if (idx < nvec) {
                float x[8];
                scaled8(v[i], inv_s, idx * 8, x);
#pragma unroll
                for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(x[e]));
            }
        }
    } else {
        for (int idx = tid; idx < nvec; idx += kActThreads) {
            float x[8];
            scaled8(__ldg(row + idx), inv_s, idx * 8, x);
#pragma unroll
            for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(x[e]));
        }
    }
    amax = block_max(amax, red);
    if (amax == 0.0f) {
        if (tid == 0) tok_scale[m] = 0.0f;
        for (int idx = tid; idx < nvec; idx += kActThreads) out[idx] = make_uint2(0u, 0u);
        return;
    }
    const float r = __fdiv_rn(127.0f, amax);
    if (tid == 0) tok_scale[m] = __fdiv_rn(amax, 127.0f);
    if (NV > 0) {
#pragma unroll
        for (int i = 0; i < NR; ++i) {
            const int idx = tid + i * kActThreads;
            if (idx < nvec) {
                float x[8];
                scaled8(v[i], inv_s, idx * 8, x);
                out[idx] = quantize8(x, r);
            }
        }
    } else {
        for (int idx = tid; idx < nvec; idx += kActThreads) {
            float x[8];
            scaled8(__ldg(row + idx), inv_s, idx * 8, x);
            out[idx] = quantize8(x, r);
        }
    }
}

// Streaming form for K <= 16384: a CTA of T = K / 16 threads (rounded up to whole warps) walks
// over tokens m = blockIdx.x, blockIdx.x + gridDim.x, ...; a thread owns the same sixteen
// features of every token, so their reciprocal scales stay in registers for the whole launch.
// In the one-token-per-CTA kernel above every element costs eight bytes of scale loads (two
// passes) from L1 next to its two bytes from HBM, and those loads, not HBM, set its speed
// (2048 x 16384: 28 us with the scale vector, 19 us without).  The next token's vectors are
// requested before the current one is reduced; the scaled values stay in registers between the
// absmax pass and the rounding pass.
template <bool SCALED>
__global__ void __launch_bounds__(1024, 1)
act_quant_stream_kernel(const __half *__restrict__ X, const float *__restrict__ inv_s, int M, int K,
                        int8_t *__restrict__ Xq, float *__restrict__ tok_scale)
{
    __shared__ float red[2][32];
    allow_dependents();
    dependent_wait();                      // X may be the output of the kernel before
    const int tid = threadIdx.x, T = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = T >> 5;
    const int nvec = K >> 3;
    const int i0 = tid, i1 = tid + T;
    const bool h0 = i0 < nvec, h1 = i1 < nvec;
    float sc[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) sc[e] = 1.0f;
    if (SCALED) {
        if (h0) {
            const float4 a = __ldg(reinterpret_cast<const float4 *>(inv_s + i0 * 8));
            const float4 b = __ldg(reinterpret_cast<const float4 *>(inv_s + i0 * 8 + 4));
            sc[0] = a.x; sc[1] = a.y; sc[2] = a.z; sc[3] = a.w;
            sc[4] = b.x; sc[5] = b.y; sc[6] = b.z; sc[7] = b.w;
        }
        if (h1) {
            const float4 a = __ldg(reinterpret_cast<const float4 *>(inv_s + i1 * 8));
            const float4 b = __ldg(reinterpret_cast<const float4 *>(inv_s + i1 * 8 + 4));
            sc[8] = a.x; sc[9] = a.y; sc[10] = a.z; sc[11] = a.w;
            sc[12] = b.x; sc[13] = b.y; sc[14] = b.z; sc[15] = b.w;
        }
    }
    const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
    int m = blockIdx.x;
    uint4 n0 = zero4, n1 = zero4;
    if (m < M) {
        const uint4 *row = reinterpret_cast<const uint4 *>(X + (size_t)m * K);
        if (h0) n0 = __ldcs(row + i0);
        if (h1) n1 = __ldcs(row + i1);
    }
    for (int it = 0; m < M; m += gridDim.x, ++it) {
        const uint4 v0 = n0, v1 = n1;
        const int mn = m + gridDim.x;
        if (mn < M) {
            const uint4 *row = reinterpret_cast<const uint4 *>(X + (size_t)mn * K);
            if (h0) n0 = __ldcs(row + i0);
            if (h1) n1 = __ldcs(row + i1);
        }
        // x' = fl(float(X) * inv_s), one rounded FP32 product per element
        float x[16];
        {
            const __half2 *p0 = reinterpret_cast<const __half2 *>(&v0);
            const __half2 *p1 = reinterpret_cast<const __half2 *>(&v1);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f0 = __half22float2(p0[i]), f1 = __half22float2(p1[i]);
                x[2 * i] = f0.x; x[2 * i + 1] = f0.y;
                x[8 + 2 * i] = f1.x; x[8 + 2 * i + 1] = f1.y;
            }
            if (SCALED) {
#pragma unroll
                for (int e = 0; e < 16; ++e) x[e] = __fmul_rn(x[e], sc[e]);
            }
        }
        float amax = 0.0f;
#pragma unroll
        for (int e = 0; e < 16; ++e) amax = fmaxf(amax, fabsf(x[e]));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        // the two halves of `red` alternate: a warp can be one barrier ahead of another, not two
        float *r2 = red[it & 1];
        if (lane == 0) r2[warp] = amax;
        __syncthreads();
        amax = lane < nwarps ? r2[lane] : 0.0f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        uint2 *out = reinterpret_cast<uint2 *>(Xq + (size_t)m * K);
        if (amax == 0.0f) {
            if (tid == 0) tok_scale[m] = 0.0f;
            if (h0) out[i0] = make_uint2(0u, 0u);
            if (h1) out[i1] = make_uint2(0u, 0u);
            continue;
        }
        const float r = __fdiv_rn(127.0f, amax);
        if (tid == 0) tok_scale[m] = __fdiv_rn(amax, 127.0f);
        uint2 q0, q1;
        q0.x = pack4(x, r); q0.y = pack4(x + 4, r);
        q1.x = pack4(x + 8, r); q1.y = pack4(x + 12, r);
        if (h0) out[i0] = q0;
        if (h1) out[i1] = q1;
    }
}

// ---------------------------------------------------------------------------
// asymmetric variant (Appendix A.1: token-wise Min-Max asymmetric quantization)
// ---------------------------------------------------------------------------
// Per token: lo = min(0, min x'), hi = max(0, max x'), d = hi - lo, step = d / 255, r = 255 / d,
// zx = clamp(rint(-lo * r), 0, 255), Q = clamp(rint(x' * r) + zx, 0, 255); stored are Q - 128
// (INT8) and zx - 128, the form the INT8 contraction takes unchanged.

__device__ __forceinline__ float2 block_min_max(float lo, float hi, float *smem)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if ((threadIdx.x & 31) == 0) {
        smem[threadIdx.x >> 5] = lo;
        smem[kActThreads / 32 + (threadIdx.x >> 5)] = hi;
    }
    __syncthreads();
    float a = smem[0], b = smem[kActThreads / 32];
#pragma unroll
    for (int w = 1; w < kActThreads / 32; ++w) {
        a = fminf(a, smem[w]);
        b = fmaxf(b, smem[kActThreads / 32 + w]);
    }
    return make_float2(a, b);
}

// rint(x * r) + zx clamped to 0..255, minus 128, as the low byte of the result: the product
// is rounded to binary32, adding 1.5 * 2^23 rounds it to an integer (half to even) in the low
// mantissa bits, and `shift` = zx - 128 - bits(1.5 * 2^23) turns those bits into the answer.
__device__ __forceinline__ uint32_t asym_bits(float x, float r, int shift)
{
    const int q = (int)__float_as_uint(__fadd_rn(__fmul_rn(x, r), 12582912.0f)) + shift;
    return (uint32_t)max(-128, min(127, q));
}

__device__ __forceinline__ uint2 quantize8_asym(const float (&x)[8], float r, int shift)
{
    uint2 o;
    o.x = prmt_b(prmt_b(asym_bits(x[0], r, shift), asym_bits(x[1], r, shift), 0x0040u),
                 prmt_b(asym_bits(x[2], r, shift), asym_bits(x[3], r, shift), 0x0040u), 0x5410u);
    o.y = prmt_b(prmt_b(asym_bits(x[4], r, shift), asym_bits(x[5], r, shift), 0x0040u),
                 prmt_b(asym_bits(x[6], r, shift), asym_bits(x[7], r, shift), 0x0040u), 0x5410u);
    return o;
}

// Streaming form of the asymmetric quantizer for K <= 16384 (see act_quant_stream_kernel: tokens
// walk through a CTA whose threads keep their sixteen reciprocal scales in registers).
template <bool SCALED>
__global__ void __launch_bounds__(1024, 1)
act_quant_asym_stream_kernel(const __half *__restrict__ X, const float *__restrict__ inv_s, int M,
                             int K, int8_t *__restrict__ Xq, float *__restrict__ tok_scale,
                             int32_t *__restrict__ tok_zero)
{
    __shared__ float red[2][64];
    allow_dependents();
    dependent_wait();                      // X may be the output of the kernel before
    const int tid = threadIdx.x, T = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = T >> 5;
    const int nvec = K >> 3;
    const int i0 = tid, i1 = tid + T;
    const bool h0 = i0 < nvec, h1 = i1 < nvec;
    float sa[8], sb[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) { sa[e] = 1.0f; sb[e] = 1.0f; }
    if (SCALED) {
        if (h0) {
            const float4 a = __ldg(reinterpret_cast<const float4 *>(inv_s + i0 * 8));
            const float4 b = __ldg(reinterpret_cast<const float4 *>(inv_s + i0 * 8 + 4));
            sa[0] = a.x; sa[1] = a.y; sa[2] = a.z; sa[3] = a.w;
            sa[4] = b.x; sa[5] = b.y; sa[6] = b.z; sa[7] = b.w;
        }
        if (h1) {
            const float4 a = __ldg(reinterpret_cast<const float4 *>(inv_s + i1 * 8));
            const float4 b = __ldg(reinterpret_cast<const float4 *>(inv_s + i1 * 8 + 4));
            sb[0] = a.x; sb[1] = a.y; sb[2] = a.z; sb[3] = a.w;
            sb[4] = b.x; sb[5] = b.y; sb[6] = b.z; sb[7] = b.w;
        }
    }
    const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
    int m = blockIdx.x;
    uint4 n0 = zero4, n1 = zero4;
    if (m < M) {
        const uint4 *row = reinterpret_cast<const uint4 *>(X + (size_t)m * K);
        if (h0) n0 = __ldcs(row + i0);
        if (h1) n1 = __ldcs(row + i1);
    }
    for (int it = 0; m < M; m += gridDim.x, ++it) {
        const uint4 v0 = n0, v1 = n1;
        const int mn = m + gridDim.x;
        if (mn < M) {
            const uint4 *row = reinterpret_cast<const uint4 *>(X + (size_t)mn * K);
            if (h0) n0 = __ldcs(row + i0);
            if (h1) n1 = __ldcs(row + i1);
        }
        float xa[8], xb[8];
        {
            const __half2 *p0 = reinterpret_cast<const __half2 *>(&v0);
            const __half2 *p1 = reinterpret_cast<const __half2 *>(&v1);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f0 = __half22float2(p0[i]), f1 = __half22float2(p1[i]);
                xa[2 * i] = f0.x; xa[2 * i + 1] = f0.y;
                xb[2 * i] = f1.x; xb[2 * i + 1] = f1.y;
            }
            if (SCALED) {
#pragma unroll
                for (int e = 0; e < 8; ++e) { xa[e] = __fmul_rn(xa[e], sa[e]); xb[e] = __fmul_rn(xb[e], sb[e]); }
            }
        }
        float lo = 0.0f, hi = 0.0f;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            lo = fminf(lo, fminf(xa[e], xb[e]));
            hi = fmaxf(hi, fmaxf(xa[e], xb[e]));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
            hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
        }
        float *r2 = red[it & 1];
        if (lane == 0) { r2[warp] = lo; r2[32 + warp] = hi; }
        __syncthreads();
        lo = lane < nwarps ? r2[lane] : 0.0f;
        hi = lane < nwarps ? r2[32 + lane] : 0.0f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
            hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
        }
        uint2 *out = reinterpret_cast<uint2 *>(Xq + (size_t)m * K);
        const float d = __fsub_rn(hi, lo);
        if (d == 0.0f) {
            // the token is all zero: codes 0 with zero-point 0, i.e. -128 in both stored forms
            if (tid == 0) { tok_scale[m] = 0.0f; tok_zero[m] = -128; }
            if (h0) out[i0] = make_uint2(0x80808080u, 0x80808080u);
            if (h1) out[i1] = make_uint2(0x80808080u, 0x80808080u);
            continue;
        }
        const float r = __fdiv_rn(255.0f, d);
        const int zx = max(0, min(255, __float2int_rn(__fmul_rn(-lo, r))));
        if (tid == 0) { tok_scale[m] = __fdiv_rn(d, 255.0f); tok_zero[m] = zx - 128; }
        const int shift = zx - 128 - 0x4B400000;
        if (h0) out[i0] = quantize8_asym(xa, r, shift);
        if (h1) out[i1] = quantize8_asym(xb, r, shift);
    }
}

template <int NV>
__global__ void __launch_bounds__(kActThreads)
act_quant_asym_kernel(const __half *__restrict__ X, const float *__restrict__ inv_s, int M, int K,
                      int8_t *__restrict__ Xq, float *__restrict__ tok_scale,
                      int32_t *__restrict__ tok_zero)
{
    __shared__ float red[2 * kActThreads / 32];
    allow_dependents();
    dependent_wait();                      // X may be the output of the kernel before
    const int m = blockIdx.x;
    const int tid = threadIdx.x;
    const int nvec = K >> 3;
    const uint4 *row = reinterpret_cast<const uint4 *>(X + (size_t)m * K);
    uint2 *out = reinterpret_cast<uint2 *>(Xq + (size_t)m * K);
    constexpr int NR = NV > 0 ? NV : 1;
    uint4 v[NR];
    float lo = 0.0f, hi = 0.0f;
    if (NV > 0) {
#pragma unroll
        for (int i = 0; i < NR; ++i) {
            const int idx = tid + i * kActThreads;
            v[i] = make_uint4(0u, 0u, 0u, 0u);
            if (idx < nvec) v[i] = __ldcs(row + idx);
        }
#pragma unroll
        for (int i = 0; i < NR; ++i) {
            const int idx = tid + i * kActThreads;
            if (idx < nvec) {
                float x[8];
                scaled8(v[i], inv_s, idx * 8, x);
#pragma unroll
                for (int e = 0; e < 8; ++e) { lo = fminf(lo, x[e]); hi = fmaxf(hi, x[e]); }
            }
        }
    } else {
        for (int idx = tid; idx < nvec; idx += kActThreads) {
            float x[8];
            scaled8(__ldg(row + idx), inv_s, idx * 8, x);
#pragma unroll
            for (int e = 0; e < 8; ++e) { lo = fminf(lo, x[e]); hi = fmaxf(hi, x[e]); }
        }
    }
    const float2 mm = block_min_max(lo, hi, red);
    const float d = __fsub_rn(mm.y, mm.x);
    if (d == 0.0f) {
        // the token is all zero: codes 0 with zero-point 0, i.e. -128 in both stored forms
        if (tid == 0) { tok_scale[m] = 0.0f; tok_zero[m] = -128; }
        for (int idx = tid; idx < nvec; idx += kActThreads) out[idx] = make_uint2(0x80808080u, 0x80808080u);
        return;
    }
    const float r = __fdiv_rn(255.0f, d);
    const int zx = max(0, min(255, __float2int_rn(__fmul_rn(-mm.x, r))));
    if (tid == 0) { tok_scale[m] = __fdiv_rn(d, 255.0f); tok_zero[m] = zx - 128; }
    const int shift = zx - 128 - 0x4B400000;
    if (NV > 0) {
#pragma unroll
        for (int i = 0; i < NR; ++i) {
            const int idx = tid + i * kActThreads;
            if (idx < nvec) {
                float x[8];
                scaled8(v[i], inv_s, idx * 8, x);
                out[idx] = quantize8_asym(x, r, shift);
            }
        }
    } else {
        for (int idx = tid; idx < nvec; idx += kActThreads) {
            float x[8];
            scaled8(__ldg(row + idx), inv_s, idx * 8, x);
            out[idx] = quantize8_asym(x, r, shift);
        }
    }
}

}  // namespace

cudaError_t launch_quantize_act(const __half *X, const float *inv_s, int M, int K, int8_t *Xq,
                                float *tok_scale, cudaStream_t st)
{
    const int nvec = K / 8;
    if (nvec <= 2048) {
        // streaming form: sixteen features per thread, as many CTAs as are resident at once
        // (64 registers per thread: 1024 threads per SM)
        const int threads = ((nvec + 1) / 2 + 31) / 32 * 32;
        const int per_sm = 1024 / threads > 0 ? 1024 / threads : 1;
        const int sms = device_sms();
        const int grid = M < sms * per_sm ? M : sms * per_sm;
        if (inv_s)
            launch_overlapped(act_quant_stream_kernel<true>, dim3(grid), dim3(threads), 0, st, X, inv_s, M, K, Xq, tok_scale);
        else
            launch_overlapped(act_quant_stream_kernel<false>, dim3(grid), dim3(threads), 0, st, X, inv_s, M, K, Xq, tok_scale);
        return cudaGetLastError();
    }
    const int per_thread = (nvec + kActThreads - 1) / kActThreads;
    if (per_thread <= 1)
        launch_overlapped(act_quant_kernel<1>, dim3(M), dim3(kActThreads), 0, st, X, inv_s, M, K, Xq, tok_scale);
    else if (per_thread <= 2)
        launch_overlapped(act_quant_kernel<2>, dim3(M), dim3(kActThreads), 0, st, X, inv_s, M, K, Xq, tok_scale);
    else if (per_thread <= 4)
        launch_overlapped(act_quant_kernel<4>, dim3(M), dim3(kActThreads), 0, st, X, inv_s, M, K, Xq, tok_scale);
    else if (per_thread <= 8)
        launch_overlapped(act_quant_kernel<8>, dim3(M), dim3(kActThreads), 0, st, X, inv_s, M, K, Xq, tok_scale);
    else
        launch_overlapped(act_quant_kernel<0>, dim3(M), dim3(kActThreads), 0, st, X, inv_s, M, K, Xq, tok_scale);
    return cudaGetLastError();
}

}  // namespace w4a8

namespace w4a8 {

cudaError_t launch_quantize_act_asym(const __half *X, const float *inv_s, int M, int K, int8_t *Xq,
                                     float *tok_scale, int32_t *tok_zero, cudaStream_t st)
{
    const int nvec = K / 8;
    if (nvec <= 2048) {
        const int threads = ((nvec + 1) / 2 + 31) / 32 * 32;
        const int per_sm = 1024 / threads > 0 ? 1024 / threads : 1;
        const int sms = device_sms();
        const int ctas = M < sms * per_sm ? M : sms * per_sm;
        if (inv_s)
            launch_overlapped(act_quant_asym_stream_kernel<true>, dim3(ctas), dim3(threads), 0, st, X, inv_s, M, K, Xq, tok_scale, tok_zero);
        else
            launch_overlapped(act_quant_asym_stream_kernel<false>, dim3(ctas), dim3(threads), 0, st, X, inv_s, M, K, Xq, tok_scale, tok_zero);
        return cudaGetLastError();
    }
    const int per_thread = (nvec + kActThreads - 1) / kActThreads;
    const dim3 grid(M), block(kActThreads);
    if (per_thread <= 1)
        launch_overlapped(act_quant_asym_kernel<1>, grid, block, 0, st, X, inv_s, M, K, Xq, tok_scale, tok_zero);
    else if (per_thread <= 2)
        launch_overlapped(act_quant_asym_kernel<2>, grid, block, 0, st, X, inv_s, M, K, Xq, tok_scale, tok_zero);
    else if (per_thread <= 4)
        launch_overlapped(act_quant_asym_kernel<4>, grid, block, 0, st, X, inv_s, M, K, Xq, tok_scale, tok_zero);
    else if (per_thread <= 8)
        launch_overlapped(act_quant_asym_kernel<8>, grid, block, 0, st, X, inv_s, M, K, Xq, tok_scale, tok_zero);
    else
        launch_overlapped(act_quant_asym_kernel<0>, grid, block, 0, st, X, inv_s, M, K, Xq, tok_scale, tok_zero);
    return cudaGetLastError();
}

}  // namespace w4a8
