// Weight packing: Q(W diag(s)) of Eq. 1 with the dINT4 quantizer of Eq. 5, written in
// the tiled blob layout, and its inverse (test export).
#include "common.cuh"

namespace w4a8 {

namespace {

constexpr int kPackThreads = 256;

// Eq. 5 for b = 4: codes 0..13 integer levels, 14 = c1 (+c), 15 = c2 (-c), c = s / 2^shift.
// A value is special between the midpoints of (0, c) and (c, s): `lower` = c / 2,
// `upper` = (c + s) / 2, i.e. s/4 and 3s/4 for the paper's c = s/2.
__device__ __forceinline__ void special_band(float s, int shift, float &lower, float &upper)
{
    lower = __fmul_rn(0.5f * level_unit(shift), s);
    upper = shift == 1 ? __fmul_rn(0.75f, s) : __fadd_rn(__fmul_rn(0.5f, s), lower);
}
__device__ __forceinline__ uint32_t dint4_quantize(float x, float s, int z, float quarter,
                                                   float threeq)
{
    if (x > quarter && x <= threeq) return 14u;
    if (x < -quarter && x >= -threeq) return 15u;
    float r = rintf(__fdiv_rn(x, s));
    r = fminf(fmaxf(r, -1048576.0f), 1048576.0f);
    int q = (int)r + z;
    q = q < 0 ? 0 : (q > 13 ? 13 : q);
    return (uint32_t)q;
}

// step = range / p and zero-point for p uniform steps (p = 13 for 4-bit codes, 5 for 3-bit)
__device__ __forceinline__ void step_and_zero(float lo, float hi, float clip, float &s, int &z,
                                              int p = 13)
{
    lo = __fmul_rn(lo, clip);
    hi = __fmul_rn(hi, clip);
    s = __fdiv_rn(__fsub_rn(hi, lo), (float)p);
    if (s == 0.0f) s = 1.0f;
    float r = rintf(__fdiv_rn(-lo, s));
    r = fminf(fmaxf(r, -1048576.0f), 1048576.0f);
    z = (int)r;
    z = z < 0 ? 0 : (z > p ? p : z);
}

// Eq. 5 for b = 3: codes 0..5 integer levels, 6 = c1 (+c), 7 = c2 (-c)
__device__ __forceinline__ uint32_t dint3_quantize(float x, float s, int z, float lower, float upper)
{
    if (x > lower && x <= upper) return 6u;
    if (x < -lower && x >= -upper) return 7u;
    float r = rintf(__fdiv_rn(x, s));
    r = fminf(fmaxf(r, -1048576.0f), 1048576.0f);
    int q = (int)r + z;
    q = q < 0 ? 0 : (q > 5 ? 5 : q);
    return (uint32_t)q;
}

__device__ __forceinline__ float scaled(const __half h, const float *s_in, int k)
{
    const float w = __half2float(h);
    return s_in ? __fmul_rn(w, s_in[k]) : w;
}

__device__ __forceinline__ void write_header(uint8_t *blob, const BlobLayout &L, float clip)
{
    BlobHeader h;
    memset(&h, 0, sizeof(h));
    h.magic = kBlobMagic;
    h.version = kBlobVersion;
    h.layout = kBlobLayoutQuarterRow16;
    h.group = (uint32_t)L.group;
    h.N = L.N; h.K = L.K; h.G = L.G;
    h.n_tiles = L.n_tiles; h.k_blocks = L.k_blocks; h.n_pad = L.n_pad;
    h.off_scales = L.off_scales; h.off_zeros = L.off_zeros;
    h.off_codes = L.off_codes; h.total_bytes = L.total_bytes;
    h.clip = clip;
    h.level_shift = (uint32_t)L.shift;
    h.bits = (uint32_t)L.bits;
    *reinterpret_cast<BlobHeader *>(blob) = h;
}

// One CTA per output row; the whole row is one quantization group.
__global__ void __launch_bounds__(kPackThreads)
pack_rows_kernel(const __half *__restrict__ W, const float *__restrict__ s_in, BlobLayout L,
                 float clip, uint8_t *__restrict__ blob)
{
    const int n = blockIdx.x;
    const int tid = threadIdx.x;
    float *scales = reinterpret_cast<float *>(blob + L.off_scales);
    uint8_t *zeros = blob + L.off_zeros;
    uint8_t *codes = blob + L.off_codes;
    if (n == 0 && tid == 0) write_header(blob, L, clip);

    __shared__ float s_lo[kPackThreads / 32], s_hi[kPackThreads / 32];
    __shared__ float s_step;
    __shared__ int s_zero;

    const bool real = n < L.N;
    const __half *row = W + (size_t)n * L.K;
    float lo = 0.0f, hi = 0.0f;
    if (real) {
        for (int k0 = tid * 8; k0 < L.K; k0 += kPackThreads * 8) {
            const uint4 v = *reinterpret_cast<const uint4 *>(row + k0);
            const __half *h = reinterpret_cast<const __half *>(&v);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float w = scaled(h[i], s_in, k0 + i);
                if (w < lo) lo = w;
                if (w > hi) hi = w;
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float l2 = __shfl_xor_sync(0xffffffffu, lo, o);
        const float h2 = __shfl_xor_sync(0xffffffffu, hi, o);
        if (l2 < lo) lo = l2;
        if (h2 > hi) hi = h2;
    }
    if ((tid & 31) == 0) { s_lo[tid >> 5] = lo; s_hi[tid >> 5] = hi; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < kPackThreads / 32; ++w) {
            if (s_lo[w] < lo) lo = s_lo[w];
            if (s_hi[w] > hi) hi = s_hi[w];
        }
        float s; int z;
        step_and_zero(lo, hi, clip, s, z);
        s_step = s; s_zero = z;
        scales[n] = s;
        zeros[n] = (uint8_t)z;
    }
    __syncthreads();
    const float s = s_step;
    const int z = s_zero;
    float quarter, threeq;
    special_band(s, L.shift, quarter, threeq);
    for (int k0 = tid * 8; k0 < L.K; k0 += kPackThreads * 8) {
        uint32_t word = 0;
        if (real) {
            const uint4 v = *reinterpret_cast<const uint4 *>(row + k0);
            const __half *h = reinterpret_cast<const __half *>(&v);
#pragma unroll
            for (int i = 0; i < 8; ++i)
                word |= dint4_quantize(scaled(h[i], s_in, k0 + i), s, z, quarter, threeq) << (4 * i);
        }
        *reinterpret_cast<uint32_t *>(codes + code_byte_offset(L, n, k0)) = word;
    }
}

// One CTA per output row; each warp takes one 128-wide group at a time.
__global__ void __launch_bounds__(kPackThreads)
pack_groups_kernel(const __half *__restrict__ W, const float *__restrict__ s_in, BlobLayout L,
                   float clip, uint8_t *__restrict__ blob)
{
    const int n = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float *scales = reinterpret_cast<float *>(blob + L.off_scales);
    uint8_t *zeros = blob + L.off_zeros;
    uint8_t *codes = blob + L.off_codes;
    if (n == 0 && threadIdx.x == 0) write_header(blob, L, clip);
    const bool real = n < L.N;
    const __half *row = W + (size_t)n * L.K;
    for (int g = warp; g < L.G; g += kPackThreads / 32) {
        const int k0 = g * 128 + lane * 4;
        float w[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        if (real) {
            const uint2 v = *reinterpret_cast<const uint2 *>(row + k0);
            const __half *h = reinterpret_cast<const __half *>(&v);
#pragma unroll
            for (int i = 0; i < 4; ++i) w[i] = scaled(h[i], s_in, k0 + i);
        }
        float lo = 0.0f, hi = 0.0f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (w[i] < lo) lo = w[i];
            if (w[i] > hi) hi = w[i];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float l2 = __shfl_xor_sync(0xffffffffu, lo, o);
            const float h2 = __shfl_xor_sync(0xffffffffu, hi, o);
            if (l2 < lo) lo = l2;
            if (h2 > hi) hi = h2;
        }
        float s; int z;
        step_and_zero(lo, hi, clip, s, z);
        if (lane == 0) {
            scales[(size_t)g * L.n_pad + n] = s;
            zeros[(size_t)g * L.n_pad + n] = (uint8_t)z;
        }
        float quarter, threeq;
        special_band(s, L.shift, quarter, threeq);
        uint32_t half_word = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i)
            half_word |= dint4_quantize(w[i], s, z, quarter, threeq) << (4 * i);
        *reinterpret_cast<uint16_t *>(codes + code_byte_offset(L, n, k0)) = (uint16_t)half_word;
    }
}

// 3-bit codes (dINT3), per-channel or group-128: one CTA of 128 threads per output row.  A
// thread takes 32-k quarters of the row; the four threads of a 128-wide chunk combine their
// ranges by shuffles, the chunks' ranges wait in shared memory (the whole row's for
// per-channel weights), then every thread re-reads its quarters and writes three words each.
__global__ void __launch_bounds__(128)
pack3_kernel(const __half *__restrict__ W, const float *__restrict__ s_in, BlobLayout L, float clip,
             uint8_t *__restrict__ blob)
{
    extern __shared__ float s_range[];               // lo[chunks], hi[chunks]
    const int n = blockIdx.x, tid = threadIdx.x;
    float *scales = reinterpret_cast<float *>(blob + L.off_scales);
    uint8_t *zeros = blob + L.off_zeros;
    uint8_t *codes = blob + L.off_codes;
    if (n == 0 && tid == 0) write_header(blob, L, clip);
    const bool real = n < L.N;
    const __half *row = W + (size_t)n * L.K;
    const int chunks = L.k_blocks, quarters = 4 * chunks;
    float *s_lo = s_range, *s_hi = s_range + chunks;
    for (int qi = tid; qi < (quarters + 127) / 128 * 128; qi += 128) {
        float lo = 0.0f, hi = 0.0f;
        if (real && qi < quarters) {
            for (int i = 0; i < 32; ++i) {
                const float w = scaled(row[qi * 32 + i], s_in, qi * 32 + i);
                if (w < lo) lo = w;
                if (w > hi) hi = w;
            }
        }
        for (int o = 1; o <= 2; o <<= 1) {
            const float l2 = __shfl_xor_sync(0xffffffffu, lo, o);
            const float h2 = __shfl_xor_sync(0xffffffffu, hi, o);
            if (l2 < lo) lo = l2;
            if (h2 > hi) hi = h2;
        }
        if ((tid & 3) == 0 && qi < quarters) { s_lo[qi >> 2] = lo; s_hi[qi >> 2] = hi; }
    }
    __syncthreads();
    if (L.group == 0) {
        if (tid == 0) {
            float lo = 0.0f, hi = 0.0f;
            for (int c = 0; c < chunks; ++c) {
                if (s_lo[c] < lo) lo = s_lo[c];
                if (s_hi[c] > hi) hi = s_hi[c];
            }
            float s; int z;
            step_and_zero(lo, hi, clip, s, z, 5);
            scales[n] = s;
            zeros[n] = (uint8_t)z;
            s_lo[0] = s;
            s_hi[0] = __int_as_float(z);
        }
    } else {
        for (int c = tid; c < chunks; c += 128) {
            float s; int z;
            step_and_zero(s_lo[c], s_hi[c], clip, s, z, 5);
            scales[(size_t)c * L.n_pad + n] = s;
            zeros[(size_t)c * L.n_pad + n] = (uint8_t)z;
            s_lo[c] = s;
            s_hi[c] = __int_as_float(z);
        }
    }
    __syncthreads();
    for (int qi = tid; qi < quarters; qi += 128) {
        const int c = L.group == 0 ? 0 : (qi >> 2);
        const float s = s_lo[c];
        const int z = __float_as_int(s_hi[c]);
        float lower, upper;
        special_band(s, L.shift, lower, upper);
        uint32_t w[3] = {0u, 0u, 0u};
        if (real) {
            for (int i = 0; i < 32; ++i) {
                const uint32_t code = dint3_quantize(scaled(row[qi * 32 + i], s_in, qi * 32 + i), s, z, lower, upper);
                if (i < 24) {
                    w[i >> 3] |= code << (4 * (i & 7));
                } else {
                    const int sh = 4 * (i - 24) + 3;
                    w[0] |= (code & 1u) << sh;
                    w[1] |= ((code >> 1) & 1u) << sh;
                    w[2] |= ((code >> 2) & 1u) << sh;
                }
            }
        }
        for (int j = 0; j < 3; ++j)
            *reinterpret_cast<uint32_t *>(codes + code3_word_offset(L, n, qi >> 2, qi & 3, j)) = w[j];
    }
}

// Per-output-channel packing of a matrix that arrives transposed, Wt[K][N] (the attention
// value tensor V[s][h * D + d]: its channels are the outputs, the sequence is the reduction
// dimension).  A CTA takes 32 consecutive channels n (lane = channel, so a warp reads 64
// contiguous bytes of a row of Wt); its 8 warps split the k range.
__global__ void __launch_bounds__(kPackThreads)
pack_transposed_kernel(const __half *__restrict__ Wt, BlobLayout L, float clip,
                       uint8_t *__restrict__ blob)
{
    __shared__ float s_lo[8][32], s_hi[8][32];
    __shared__ float s_step[32];
    __shared__ int s_zero[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n = blockIdx.x * 32 + lane;
    float *scales = reinterpret_cast<float *>(blob + L.off_scales);
    uint8_t *zeros = blob + L.off_zeros;
    uint8_t *codes = blob + L.off_codes;
    if (blockIdx.x == 0 && threadIdx.x == 0) write_header(blob, L, clip);
    const bool real = n < L.N;
    float lo = 0.0f, hi = 0.0f;
    if (real) {
        for (int k = warp; k < L.K; k += 8) {
            const float w = __half2float(Wt[(size_t)k * L.N + n]);
            if (w < lo) lo = w;
            if (w > hi) hi = w;
        }
    }
    s_lo[warp][lane] = lo;
    s_hi[warp][lane] = hi;
    __syncthreads();
    if (warp == 0) {
        for (int w = 1; w < 8; ++w) {
            if (s_lo[w][lane] < lo) lo = s_lo[w][lane];
            if (s_hi[w][lane] > hi) hi = s_hi[w][lane];
        }
        float s; int z;
        step_and_zero(lo, hi, clip, s, z);
        s_step[lane] = s;
        s_zero[lane] = z;
        if (n < L.n_pad) { scales[n] = s; zeros[n] = (uint8_t)z; }
    }
    __syncthreads();
    const float s = s_step[lane];
    const int z = s_zero[lane];
    float quarter, threeq;
    special_band(s, L.shift, quarter, threeq);
    if (n >= L.n_pad) return;
    for (int k = 2 * warp; k < L.K; k += 16) {
        uint32_t byte = 0;
        if (real) {
            const float w0 = __half2float(Wt[(size_t)k * L.N + n]);
            const float w1 = __half2float(Wt[(size_t)(k + 1) * L.N + n]);
            byte = dint4_quantize(w0, s, z, quarter, threeq) | (dint4_quantize(w1, s, z, quarter, threeq) << 4);
        }
        codes[code_byte_offset(L, n, k)] = (uint8_t)byte;
    }
}

__global__ void unpack_kernel(const uint8_t *__restrict__ blob, BlobLayout L,
                              uint8_t *__restrict__ out_codes, float *__restrict__ out_scales,
                              uint8_t *__restrict__ out_zeros)
{
    const size_t half_k = (size_t)L.K / 2;
    const size_t total = (size_t)L.N * half_k;
    const float *scales = reinterpret_cast<const float *>(blob + L.off_scales);
    const uint8_t *zeros = blob + L.off_zeros;
    const uint8_t *codes = blob + L.off_codes;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (size_t)gridDim.x * blockDim.x) {
        const int n = (int)(i / half_k);
        const int k = (int)(i % half_k) * 2;
        if (L.bits == 3) {
            const int kb = k / kTileK, q = (k % kTileK) / 32, j = k % 32;
            const uint32_t w0 = *reinterpret_cast<const uint32_t *>(codes + code3_word_offset(L, n, kb, q, 0));
            const uint32_t w1 = *reinterpret_cast<const uint32_t *>(codes + code3_word_offset(L, n, kb, q, 1));
            const uint32_t w2 = *reinterpret_cast<const uint32_t *>(codes + code3_word_offset(L, n, kb, q, 2));
            out_codes[i] = (uint8_t)(code3_of(w0, w1, w2, j) | (code3_of(w0, w1, w2, j + 1) << 4));
            continue;
        }
        out_codes[i] = codes[code_byte_offset(L, n, k)];
    }
    const size_t meta = (size_t)L.G * L.N;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < meta;
         i += (size_t)gridDim.x * blockDim.x) {
        const int g = (int)(i / L.N), n = (int)(i % L.N);
        out_scales[i] = scales[(size_t)g * L.n_pad + n];
        out_zeros[i] = zeros[(size_t)g * L.n_pad + n];
    }
}

// rowsum[g][n] = sum over the k of group g of t2(code[n][k]) (Eq. 6 in units of step/2): the
// factor of a token's zero-point in the asymmetric-activation path.  One CTA per 128-row tile
// and K slice, one thread per row; a warp reads 512 contiguous bytes per quarter tile.
// Per-channel weights: the slices add into rowsum[n] (zeroed by the launcher) with integer
// atomics, so the result does not depend on their order.  Group mode: a slice is one k-block
// and owns its entry.
__global__ void __launch_bounds__(128)
rowsum_kernel(const uint8_t *__restrict__ blob, BlobLayout L, int kb_per_slice,
              int32_t *__restrict__ rowsum)
{
    const int nt = blockIdx.x, r = threadIdx.x;
    const int n = nt * kTileN + r;
    const uint8_t *zeros = blob + L.off_zeros;
    const uint8_t *codes = blob + L.off_codes;
    // the unit of the levels is the blob's own (0 in the header of an older blob means 1)
    const uint32_t hs = reinterpret_cast<const BlobHeader *>(blob)->level_shift;
    const int shift = hs == 0u ? 1 : (int)hs;
    const int kb0 = blockIdx.y * kb_per_slice;
    const int kb1 = min(L.k_blocks, kb0 + kb_per_slice);
    int z = zeros[n];
    int sum = 0;
    for (int kb = kb0; kb < kb1; ++kb) {
        if (L.group != 0) { z = zeros[(size_t)kb * L.n_pad + n]; sum = 0; }
        const uint8_t *tile = codes + ((size_t)nt * L.k_blocks + kb) * kTileBytes;
        for (int q = 0; q < 4; ++q) {
            const uint4 w = *reinterpret_cast<const uint4 *>(tile + q * kQuarterBytes + r * 16);
            const uint32_t words[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int i = 0; i < 32; ++i) sum += dint4_level((words[i >> 3] >> (4 * (i & 7))) & 15, z, shift);
        }
        if (L.group != 0 && n < L.N) rowsum[(size_t)kb * L.N + n] = sum;
    }
    if (L.group == 0 && n < L.N) atomicAdd(rowsum + n, sum);
}

}  // namespace

cudaError_t launch_pack(const __half *W, const float *s_in, const BlobLayout &L, float clip,
                        uint8_t *blob, cudaStream_t st)
{
    if (L.bits == 3)
        pack3_kernel<<<L.n_pad, 128, 2 * L.k_blocks * sizeof(float), st>>>(W, s_in, L, clip, blob);
    else if (L.group == 0)
        pack_rows_kernel<<<L.n_pad, kPackThreads, 0, st>>>(W, s_in, L, clip, blob);
    else
        pack_groups_kernel<<<L.n_pad, kPackThreads, 0, st>>>(W, s_in, L, clip, blob);
    return cudaGetLastError();
}

cudaError_t launch_pack_transposed(const __half *Wt, const BlobLayout &L, float clip, uint8_t *blob,
                                   cudaStream_t st)
{
    pack_transposed_kernel<<<L.n_pad / 32, kPackThreads, 0, st>>>(Wt, L, clip, blob);
    return cudaGetLastError();
}

cudaError_t launch_unpack(const uint8_t *blob, const BlobLayout &L, uint8_t *codes,
                          float *scales, uint8_t *zeros, cudaStream_t st)
{
    const size_t total = (size_t)L.N * L.K / 2;
    int blocks = (int)((total + 255) / 256);
    const int cap = device_sms() * 16;
    if (blocks > cap) blocks = cap;
    unpack_kernel<<<blocks, 256, 0, st>>>(blob, L, codes, scales, zeros);
    return cudaGetLastError();
}

cudaError_t launch_weight_rowsum(const uint8_t *blob, const BlobLayout &L, int32_t *rowsum,
                                 cudaStream_t st)
{
    // enough CTAs to fill the GPU: K slices of at least one k-block
    int slices = 1;
    if (L.group != 0) {
        slices = L.k_blocks;
    } else {
        slices = (8 * device_sms() + L.n_tiles - 1) / L.n_tiles;
        if (slices > L.k_blocks) slices = L.k_blocks;
        if (cudaMemsetAsync(rowsum, 0, (size_t)L.N * sizeof(int32_t), st) != cudaSuccess)
            return cudaGetLastError();
    }
    const int per = (L.k_blocks + slices - 1) / slices;
    slices = (L.k_blocks + per - 1) / per;
    if (slices > 65535) return cudaErrorInvalidValue;
    rowsum_kernel<<<dim3(L.n_tiles, slices), 128, 0, st>>>(blob, L, per, rowsum);
    return cudaGetLastError();
}

}  // namespace w4a8
