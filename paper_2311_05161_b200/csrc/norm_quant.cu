// Token-wise INT8 activation quantizer fused with the normalisation in front of it.
//
// Eq. 1 multiplies the activations by diag(s)^-1; in a decoder layer that factor is merged
// into the weight (and bias) of the LayerNorm / RMSNorm that feeds the matmul (Fig. 1(a),
// Section 3.1), so the matmul's INT8 input is Q(norm(X)) and the normalised FP16 tensor never
// has to exist in memory: this kernel reads X once (2 bytes per element) and writes the INT8
// codes (1 byte) and the token steps, where normalisation followed by w4a8_quantize_act
// would move 2 + 2 + 2 + 1 bytes.
//
// Arithmetic (the statement the CPU checker follows too): a sum over the features is taken in
// binary32 inside each run of 8 consecutive features (one 16-byte vector; the squares enter by
// fused multiply-add, and a binary16 value squared is exact in binary32) and in binary64 across
// the runs; mean, mean square and r = 1 / sqrt(. + eps) are binary64, mean and r are rounded
// once to binary32, and x' = ((x - mean) * r) * weight (+ bias) is binary32 with one rounding
// per operation; then amax, step = amax / 127 and q = clamp(rint(x' * (127 / amax))) as in the
// stand-alone quantizer.  The binary64 partial sums are added in the kernel's own order (thread,
// warp butterfly, CTA), which can differ from an ascending sum by a few units of 2^-53: mean or
// r change only if that lands on a binary32 rounding boundary.
//
// Layout of the work: as act_quant_stream_kernel - a CTA of K / 16 threads walks over
// tokens, a thread owns the same sixteen features of every token and keeps their weights in
// registers, the next token's two 16-byte vectors are requested before the current one is
// reduced.  K <= 16384.
#include "common.cuh"
#include "quant_math.cuh"

namespace w4a8 {

namespace {

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = __dadd_rn(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Sum over the CTA; every thread gets the same value.  `buf` holds one slot per warp and must
// not be reused before another barrier has passed.
__device__ __forceinline__ double cta_sum(double v, double *buf, int lane, int warp, int nwarps)
{
    v = warp_sum(v);
    if (lane == 0) buf[warp] = v;
    __syncthreads();
    v = lane < nwarps ? buf[lane] : 0.0;
    return warp_sum(v);
}

__device__ __forceinline__ void unpack16(const uint4 &v0, const uint4 &v1, float (&x)[16])
{
    const __half2 *p0 = reinterpret_cast<const __half2 *>(&v0);
    const __half2 *p1 = reinterpret_cast<const __half2 *>(&v1);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f0 = __half22float2(p0[i]), f1 = __half22float2(p1[i]);
        x[2 * i] = f0.x; x[2 * i + 1] = f0.y;
        x[8 + 2 * i] = f1.x; x[8 + 2 * i + 1] = f1.y;
    }
}

__device__ __forceinline__ void load8(const float *p, float *dst)
{
    const float4 a = __ldg(reinterpret_cast<const float4 *>(p));
    const float4 b = __ldg(reinterpret_cast<const float4 *>(p + 4));
    dst[0] = a.x; dst[1] = a.y; dst[2] = a.z; dst[3] = a.w;
    dst[4] = b.x; dst[5] = b.y; dst[6] = b.z; dst[7] = b.w;
}

// LAYER: LayerNorm (mean removed), else RMSNorm.  BIAS: a bias vector is added.
template <bool LAYER, bool BIAS>
__global__ void __launch_bounds__(1024, 1)
norm_quant_stream_kernel(const __half *__restrict__ X, const float *__restrict__ weight,
                         const float *__restrict__ bias, float eps, int M, int K,
                         int8_t *__restrict__ Xq, float *__restrict__ tok_scale)
{
    __shared__ double red_sum[2][32], red_sq[2][32];
    __shared__ float red_max[2][32];
    allow_dependents();
    dependent_wait();                      // X may be the output of the kernel before
    const int tid = threadIdx.x, T = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarps = T >> 5;
    const int nvec = K >> 3;
    const int i0 = tid, i1 = tid + T;
    const bool h0 = i0 < nvec, h1 = i1 < nvec;
    float w[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) w[e] = 0.0f;
    if (h0) load8(weight + i0 * 8, w);
    if (h1) load8(weight + i1 * 8, w + 8);
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
        float x[16];
        unpack16(v0, v1, x);
        // ---- statistics: binary32 inside a vector of 8 features, binary64 across vectors
        // (vectors past K hold zeros and are left out) ----
        if (LAYER) {
            float p0 = 0.0f, p1 = 0.0f;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                p0 = __fadd_rn(p0, x[e]);
                p1 = __fadd_rn(p1, x[8 + e]);
            }
            double s = __dadd_rn((double)p0, (double)p1);
            s = cta_sum(s, red_sum[it & 1], lane, warp, nwarps);
            const float mu = __double2float_rn(__ddiv_rn(s, (double)K));
#pragma unroll
            for (int e = 0; e < 16; ++e) x[e] = __fsub_rn(x[e], mu);
        }
        float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            s0 = __fmaf_rn(x[e], x[e], s0);
            s1 = __fmaf_rn(x[8 + e], x[8 + e], s1);
        }
        double sq = __dadd_rn(h0 ? (double)s0 : 0.0, h1 ? (double)s1 : 0.0);
        sq = cta_sum(sq, red_sq[it & 1], lane, warp, nwarps);
        const float r = __double2float_rn(
            __ddiv_rn(1.0, __dsqrt_rn(__dadd_rn(__ddiv_rn(sq, (double)K), (double)eps))));
        // ---- x' = ((x - mean) * r) * weight (+ bias), binary32 ----
        float b[16];
        if (BIAS) {
#pragma unroll
            for (int e = 0; e < 16; ++e) b[e] = 0.0f;
            if (h0) load8(bias + i0 * 8, b);
            if (h1) load8(bias + i1 * 8, b + 8);
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            float t = __fmul_rn(__fmul_rn(x[e], r), w[e]);
            if (BIAS) t = __fadd_rn(t, b[e]);
            x[e] = t;
        }
        float amax = 0.0f;
#pragma unroll
        for (int e = 0; e < 16; ++e) amax = fmaxf(amax, fabsf(x[e]));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        float *r2 = red_max[it & 1];
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
        const float q = __fdiv_rn(127.0f, amax);
        if (tid == 0) tok_scale[m] = __fdiv_rn(amax, 127.0f);
        uint2 q0, q1;
        q0.x = pack4(x, q); q0.y = pack4(x + 4, q);
        q1.x = pack4(x + 8, q); q1.y = pack4(x + 12, q);
        if (h0) out[i0] = q0;
        if (h1) out[i1] = q1;
    }
}

}  // namespace

cudaError_t launch_norm_quantize_act(const __half *X, const float *weight, const float *bias,
                                     int layer_norm, float eps, int M, int K, int8_t *Xq,
                                     float *tok_scale, cudaStream_t st)
{
    const int nvec = K / 8;
    if (nvec > 2048) return cudaErrorInvalidValue;
    const int threads = ((nvec + 1) / 2 + 31) / 32 * 32;
    const int per_sm = 1024 / threads > 0 ? 1024 / threads : 1;
    const int sms = device_sms();
    const dim3 grid(M < sms * per_sm ? M : sms * per_sm), block(threads);
    if (layer_norm) {
        if (bias) launch_overlapped(norm_quant_stream_kernel<true, true>, grid, block, 0, st, X, weight, bias, eps, M, K, Xq, tok_scale);
        else launch_overlapped(norm_quant_stream_kernel<true, false>, grid, block, 0, st, X, weight, bias, eps, M, K, Xq, tok_scale);
    } else {
        if (bias) launch_overlapped(norm_quant_stream_kernel<false, true>, grid, block, 0, st, X, weight, bias, eps, M, K, Xq, tok_scale);
        else launch_overlapped(norm_quant_stream_kernel<false, false>, grid, block, 0, st, X, weight, bias, eps, M, K, Xq, tok_scale);
    }
    return cudaGetLastError();
}

}  // namespace w4a8
