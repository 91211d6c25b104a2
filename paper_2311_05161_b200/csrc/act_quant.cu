// Token-wise INT8 activation quantizer: Q(diag(s)^-1 X) of Eq. 1 (Appendix A.1,
// "token-wise quantization for activations"), symmetric absmax variant.
// One CTA per token; the token stays in registers between the absmax pass and the
// rounding pass, so HBM sees 2 bytes read and 1 byte written per element.
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
