// Plain CUDA-core version of the quantized linear layer: one thread per output element.
// It exists as an independent on-device cross-check of the tensor-core kernel and is
// only reached through an explicit path option; it is far too slow for real use.
#include "common.cuh"

namespace w4a8 {

namespace {

__global__ void __launch_bounds__(128)
linear_simple_kernel(const int8_t *__restrict__ Xq, const float *__restrict__ tok_scale,
                     const uint8_t *__restrict__ blob, BlobLayout L,
                     const float *__restrict__ bias, int M, __nv_bfloat16 *__restrict__ Y,
                     int32_t *__restrict__ acc_out, StatusBlock *sb, ZeroPoint zp)
{
    if (!header_matches(blob, L)) {
        if (threadIdx.x == 0) report_failure(sb, W4A8_ERR_BAD_BLOB, 1);
        return;
    }
    const int nt = blockIdx.x, r = threadIdx.x, m = blockIdx.y;
    const int n = nt * kTileN + r;
    const float *scales = reinterpret_cast<const float *>(blob + L.off_scales);
    const uint8_t *zeros = blob + L.off_zeros;
    const uint8_t *codes = blob + L.off_codes;
    const int8_t *x = Xq + (size_t)m * L.K;
    const bool grouped = L.group != 0;
    int z = zeros[n];
    int32_t acc = 0;
    float u = 0.0f;
    for (int kb = 0; kb < L.k_blocks; ++kb) {
        if (grouped) { z = zeros[(size_t)kb * L.n_pad + n]; acc = 0; }
        const uint8_t *tile = codes + ((size_t)nt * L.k_blocks + kb) * L.tile_bytes;
        for (int q = 0; q < 4; ++q) {
            if (L.bits == 3) {
                const uint32_t *w3 = reinterpret_cast<const uint32_t *>(tile + q * kQuarterBytes3 + r * 4);
                const uint32_t w0 = w3[0], w1 = w3[128], w2 = w3[256];
                const int8_t *xk = x + kb * kTileK + q * 32;
                for (int i = 0; i < 32; ++i)
                    acc += (int32_t)xk[i] * dint_level(code3_of(w0, w1, w2, i), z, L.shift, 3);
                continue;
            }
            const uint4 w = *reinterpret_cast<const uint4 *>(tile + q * kQuarterBytes + r * 16);
            const uint32_t words[4] = {w.x, w.y, w.z, w.w};
            const int8_t *xk = x + kb * kTileK + q * 32;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int code = (words[i >> 3] >> (4 * (i & 7))) & 15;
                acc += (int32_t)xk[i] * dint4_level(code, z, L.shift);
            }
        }
        if (grouped && n < L.N) {
            if (zp.tok_zero) acc -= zp.tok_zero[m] * zp.rowsum[(size_t)kb * L.N + n];
            if (acc_out) acc_out[((size_t)kb * M + m) * L.N + n] = acc;
            u = fmaf((float)acc, __fmul_rn(level_unit(L.shift), scales[(size_t)kb * L.n_pad + n]), u);
        }
    }
    if (n >= L.N) return;
    const float a = tok_scale ? tok_scale[m] : 0.0f;
    float t;
    if (grouped) {
        t = __fmul_rn(u, a);
    } else {
        if (zp.tok_zero) acc -= zp.tok_zero[m] * zp.rowsum[n];
        if (acc_out) acc_out[(size_t)m * L.N + n] = acc;
        t = rescale_channel(acc, a, __fmul_rn(level_unit(L.shift), scales[n]));
    }
    if (Y) Y[(size_t)m * L.N + n] = __float2bfloat16_rn(add_bias(t, bias, n));
}

}  // namespace

cudaError_t launch_linear_simple(const int8_t *Xq, const float *tok_scale, const uint8_t *blob,
                                 const BlobLayout &L, const float *bias, int M,
                                 __nv_bfloat16 *Y, int32_t *acc, StatusBlock *sb,
                                 cudaStream_t st, ZeroPoint zp)
{
    if (M > 65535) return cudaErrorInvalidValue;
    dim3 grid(L.n_tiles, M);
    linear_simple_kernel<<<grid, 128, 0, st>>>(Xq, tok_scale, blob, L, bias, M, Y, acc, sb, zp);
    return cudaGetLastError();
}

}  // namespace w4a8
