// Weight-streaming kernel of the W4A8-dINT linear layer for one to four tokens (decode).
//
// With so few tokens the layer is a scan of the packed weights: 0.5 byte per weight from HBM,
// about two integer instructions per weight on the CUDA cores, nothing for the tensor cores to
// win.  One CTA of 128 threads takes one 128-row tile and a K slice of two to eight 128-wide
// k-blocks of it; thread r owns output row r, loads its codes two k-blocks (128 bytes) at a
// time, one step ahead of the arithmetic, expands eight codes at a time through the same 16-entry byte table as the
// tensor-core kernel (Eq. 6 in units of step/2) and accumulates with dp4a against the INT8 tokens
// held in shared memory.  K slices leave partial sums in the workspace; the last slice of a row
// tile to finish (an atomic counter, nobody waits) adds them in slice order and applies the
// FP32 rescale, so results do not depend on scheduling.
//
// Wide layers take the row-slab variant further down instead (a CTA owns 32 rows over all of K,
// its warps split the k-blocks, nothing goes through global memory).  Both kernels expand the
// codes with the offset tables described at build_offset_tables (the 16-lane logic pipe that
// runs the permutes is what bounds them, not HBM), and both can quantize their one to four
// FP16 tokens themselves (w4a8_quantize_linear), which saves the quantizer's launch.
#include <atomic>

#include "common.cuh"
#include "decode.cuh"
#include "quant_math.cuh"

namespace w4a8 {

namespace {

constexpr int kGemvKb = 2;          // k-blocks per pipeline step (128 bytes of codes per thread)
constexpr int kGemvMaxSteps = 8;    // steps per CTA: a K slice is at most 16 k-blocks
constexpr int kGemvDepth = 2;       // steps of codes in flight per thread (asynchronous copies)
constexpr int kGemvRingBytes = kGemvDepth * kGemvKb * 4 * 128 * 16;   // 32 KiB per CTA
constexpr int kGemvMaxTokens = 4;
constexpr int kMaxGemvDevices = 64;

// One k-block (128 input features) of one output row against MT tokens: w = the row's 64 bytes
// of codes, xk = the tokens' INT8 values of this k-block (token stride in bytes).
template <int MT>
__device__ __forceinline__ void block_dot_offset(const uint4 (&w)[4], const uint32_t (&t)[4],
                                                 const int8_t *xk, size_t token_stride,
                                                 int (&acc)[MT])
{
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const uint32_t words[4] = {w[q].x, w[q].y, w[q].z, w[q].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t wv = words[i], wx = wv ^ 0x88888888u;
            const uint32_t a0 = prmt(t[0], t[1], wv), b0 = prmt(t[2], t[3], wx);
            const uint32_t a1 = prmt(t[0], t[1], wv >> 16), b1 = prmt(t[2], t[3], wx >> 16);
            if (MT == 1) {
                const uint2 x = *reinterpret_cast<const uint2 *>(xk + q * 32 + i * 8);
                acc[0] = __dp4a((int)a0, (int)x.x, acc[0]);
                acc[0] = __dp4a((int)b0, (int)x.x, acc[0]);
                acc[0] = __dp4a((int)a1, (int)x.y, acc[0]);
                acc[0] = __dp4a((int)b1, (int)x.y, acc[0]);
            } else {
                const uint32_t d0 = a0 | b0, d1 = a1 | b1;
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    const uint2 x = *reinterpret_cast<const uint2 *>(xk + m * token_stride + q * 32 + i * 8);
                    acc[m] = __dp4a((int)d0, (int)x.x, acc[m]);
                    acc[m] = __dp4a((int)d1, (int)x.y, acc[m]);
                }
            }
        }
    }
}

// Sum of the 128 INT8 values at xk, by one warp; every lane gets it.
__device__ __forceinline__ int warp_sum128(const int8_t *xk)
{
    int s = __dp4a(0x01010101, reinterpret_cast<const int *>(xk)[threadIdx.x & 31], 0);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    return s;
}

struct GemvParams {
    const uint8_t *blob;
    const uint8_t *codes;
    const float *scales;
    const uint8_t *zeros;
    const int8_t *Xq;
    const float *tok_scale;
    // Fused form (X != NULL): the tokens arrive as FP16 with the Eq. 1 reciprocal scale and
    // every CTA quantizes them itself (Xq and tok_scale are then unused).
    const __half *X;
    const float *inv_s;
    const float *bias;
    __nv_bfloat16 *Y;
    int32_t *acc_out;
    StatusBlock *sb;
    int *counters;
    void *partials;
    BlobLayout L;
    int M, slices, kb_per_slice;
    ZeroPoint zp;
    LevelTables lt;
    float unit;          // level unit as a factor of the step: 2^-shift
};


// Token-wise absmax of the scaled tokens over the whole of K (activation side of Eq. 1), by
// all threads of the CTA; the result is the same in every thread.  `red` holds warps x MT
// floats.  Same arithmetic, element by element, as the stand-alone quantizer kernel.
template <int MT>
__device__ __forceinline__ void cta_token_absmax(const __half *X, const float *inv_s, int M, int K,
                                                 float *red, float (&amax)[MT])
{
    const int nvec = K >> 3, nthr = blockDim.x, warps = nthr >> 5;
#pragma unroll
    for (int m = 0; m < MT; ++m) amax[m] = 0.0f;
#pragma unroll 2
    for (int c = threadIdx.x; c < nvec; c += nthr) {
#pragma unroll
        for (int m = 0; m < MT; ++m)
            if (m < M) {
                float x[8];
                scaled8(__ldg(reinterpret_cast<const uint4 *>(X + (size_t)m * K) + c), inv_s, c * 8, x);
#pragma unroll
                for (int e = 0; e < 8; ++e) amax[m] = fmaxf(amax[m], fabsf(x[e]));
            }
    }
#pragma unroll
    for (int m = 0; m < MT; ++m) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax[m] = fmaxf(amax[m], __shfl_xor_sync(0xffffffffu, amax[m], o));
        if ((threadIdx.x & 31) == 0) red[(threadIdx.x >> 5) * MT + m] = amax[m];
    }
    __syncthreads();
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        float a = red[m];
        for (int w = 1; w < warps; ++w) a = fmaxf(a, red[w * MT + m]);
        amax[m] = a;
    }
}

// Eight scaled elements of token m starting at feature 8 c, rounded to INT8 with the token's
// factor r = 127 / amax (0 for an all-zero token, whose codes are all zero).
__device__ __forceinline__ uint2 quantize_vec8(const __half *X, const float *inv_s, int K, int m,
                                               int c, float r)
{
    float x[8];
    scaled8(__ldg(reinterpret_cast<const uint4 *>(X + (size_t)m * K) + c), inv_s, c * 8, x);
    return quantize8(x, r);
}

template <int MT, bool GROUPED>
__global__ void __launch_bounds__(128, 6)
linear_gemv_kernel(const GemvParams P)
{
    // dynamic shared memory: the code ring, then the tokens of the K slice
    extern __shared__ __align__(16) uint8_t gemv_smem[];
    uint4 *ring = reinterpret_cast<uint4 *>(gemv_smem);
    int8_t (*s_x)[kGemvMaxSteps * kGemvKb * kTileK] =
        reinterpret_cast<int8_t (*)[kGemvMaxSteps * kGemvKb * kTileK]>(gemv_smem + kGemvRingBytes);
    __shared__ int s_last;
    __shared__ float s_amax[4 * MT];
    __shared__ float s_tok[MT];          // token steps (read or, in the fused form, computed here)
    __shared__ int s_sum[MT][kGemvMaxSteps * kGemvKb];   // sums of the tokens' values per k-block
    allow_dependents();
    const int nt = blockIdx.x, slice = blockIdx.y, r = threadIdx.x;
    const int n = nt * kTileN + r;
    const int kb_first = slice * P.kb_per_slice;
    const int kb_count = min(P.kb_per_slice, P.L.k_blocks - kb_first);
    const int steps = (kb_count + kGemvKb - 1) / kGemvKb;

    // The codes are the long-latency part.  Every thread copies its own 16-byte pieces
    // asynchronously into a private ring in shared memory, kGemvDepth steps ahead of the
    // arithmetic (256 bytes in flight per thread, no registers held, no cross-thread hand-off).
    const uint8_t *src = P.codes + ((size_t)nt * P.L.k_blocks + kb_first) * kTileBytes + r * 16;
    auto issue = [&](int step) {
        if (step < steps) {
#pragma unroll
            for (int b = 0; b < kGemvKb; ++b)
                if (step * kGemvKb + b < kb_count) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(
                            ring + (((step % kGemvDepth) * kGemvKb + b) * 4 + q) * 128 + r);
                        const uint8_t *g = src + (size_t)(step * kGemvKb + b) * kTileBytes +
                                           q * kQuarterBytes;
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(g)
                                     : "memory");
                    }
                }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");     // one group per step, even if empty
    };
    // Before the wait only prefetch hints are allowed: ask L2 for the codes of the first
    // kGemvDepth steps (contiguous tiles of this row tile), so that their HBM round trip overlaps
    // the tail of the kernel before.
    {
        const int ahead = min(kb_count, kGemvDepth * kGemvKb) * (kTileBytes / 128);
        const uint8_t *first = P.codes + ((size_t)nt * P.L.k_blocks + kb_first) * kTileBytes;
        for (int i = r; i < ahead; i += 128)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(first + (size_t)i * 128));
    }
    // earlier work in the stream (the activation quantizer, a previous call's use of the
    // workspace) is complete from here on
    dependent_wait();
#pragma unroll
    for (int s = 0; s < kGemvDepth; ++s) issue(s);
    // The header is checked while the first codes are on their way (the copies stay inside
    // the blob the caller described whatever the header says); nothing is written before it.
    if (!header_matches(P.blob, P.L)) {
        if (threadIdx.x == 0) report_failure(P.sb, W4A8_ERR_BAD_BLOB, 3);
        asm volatile("cp.async.wait_all;" ::: "memory");
        return;
    }
    // tokens of this K slice: MT rows of kb_count * 128 INT8
    if (P.X) {
        // fused form: the absmax needs the whole token, the codes only this slice
        float amax[MT];
        cta_token_absmax<MT>(P.X, P.inv_s, P.M, P.L.K, s_amax, amax);
        float rq[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            rq[m] = amax[m] > 0.0f ? __fdiv_rn(127.0f, amax[m]) : 0.0f;
            if (r == 0) s_tok[m] = amax[m] > 0.0f ? __fdiv_rn(amax[m], 127.0f) : 0.0f;
        }
        constexpr int kRowVecs = kGemvMaxSteps * kGemvKb * (kTileK / 8);
        for (int c = r; c < kRowVecs; c += 128) {
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                uint2 v = make_uint2(0u, 0u);
                if (m < P.M && c < kb_count * (kTileK / 8))
                    v = quantize_vec8(P.X, P.inv_s, P.L.K, m, kb_first * (kTileK / 8) + c, rq[m]);
                reinterpret_cast<uint2 *>(&s_x[m][0])[c] = v;
            }
        }
    } else {
        if (r < MT) s_tok[r] = (P.tok_scale && r < P.M) ? P.tok_scale[r] : 0.0f;
        constexpr int kRowChunks = kGemvMaxSteps * kGemvKb * (kTileK / 16);
        for (int i = r; i < MT * kRowChunks; i += 128) {
            const int m = i / kRowChunks, c = i % kRowChunks;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (m < P.M && c < kb_count * (kTileK / 16))
                v = __ldg(reinterpret_cast<const uint4 *>(P.Xq + (size_t)m * P.L.K + kb_first * kTileK) + c);
            reinterpret_cast<uint4 *>(&s_x[m][0])[c] = v;
        }
    }
    __syncthreads();
    // offset-table expansion (see build_offset_tables) for special values step/2 and step/4
    const bool offset_tables = P.L.shift <= 2;
    const int off = 13 << P.L.shift;
    if (offset_tables) {
        for (int i = r >> 5; i < MT * kb_count; i += 4) {
            const int m = i / kb_count, kl = i - m * kb_count;
            const int sum = warp_sum128(&s_x[m][kl * kTileK]);
            if ((r & 31) == 0) s_sum[m][kl] = sum;
        }
        __syncthreads();
    }

    int acc[MT];
    float usum[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) { acc[m] = 0; usum[m] = 0.0f; }
    uint32_t t[4];
    if (!GROUPED) {
        if (offset_tables) build_offset_tables(P.zeros[n], P.lt, P.L.shift, t);
        else build_level_tables(P.zeros[n], P.lt, t);
    }
#pragma unroll 1
    for (int step = 0; step < steps; ++step) {
        // the group of this step is the oldest of kGemvDepth outstanding ones
        asm volatile("cp.async.wait_group %0;" ::"n"(kGemvDepth - 1) : "memory");
        uint4 w[kGemvKb][4];
#pragma unroll
        for (int b = 0; b < kGemvKb; ++b)
#pragma unroll
            for (int q = 0; q < 4; ++q)
                w[b][q] = ring[(((step % kGemvDepth) * kGemvKb + b) * 4 + q) * 128 + r];
        issue(step + kGemvDepth);                            // refill the slot just read
#pragma unroll
        for (int b = 0; b < kGemvKb; ++b) {
            const int kl = step * kGemvKb + b;             // k-block inside the slice
            if (kl < kb_count) {
                const int kb = kb_first + kl;
                if (GROUPED) {
                    const int z = P.zeros[(size_t)kb * P.L.n_pad + n];
                    if (offset_tables) build_offset_tables(z, P.lt, P.L.shift, t);
                    else build_level_tables(z, P.lt, t);
#pragma unroll
                    for (int m = 0; m < MT; ++m) acc[m] = 0;
                }
                if (offset_tables) {
                    block_dot_offset<MT>(w[b], t, &s_x[0][kl * kTileK], sizeof(s_x[0]), acc);
#pragma unroll
                    for (int m = 0; m < MT; ++m) acc[m] = (int)((uint32_t)acc[m] - (uint32_t)off * (uint32_t)s_sum[m][kl]);
                } else {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const uint32_t words[4] = {w[b][q].x, w[b][q].y, w[b][q].z, w[b][q].w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint32_t d0, d1;
                            decode8(words[i], t, d0, d1);
#pragma unroll
                            for (int m = 0; m < MT; ++m) {
                                const uint2 x = *reinterpret_cast<const uint2 *>(
                                    &s_x[m][kl * kTileK + q * 32 + i * 8]);
                                acc[m] = __dp4a((int)d0, (int)x.x, acc[m]);
                                acc[m] = __dp4a((int)d1, (int)x.y, acc[m]);
                            }
                        }
                    }
                }
                if (GROUPED) {
                    const float h = __fmul_rn(P.unit, P.scales[(size_t)kb * P.L.n_pad + n]);
                    // asymmetric activations: the token's zero-point times this group's level sum
                    const int rs = (P.zp.tok_zero && n < P.L.N) ? P.zp.rowsum[(size_t)kb * P.L.N + n] : 0;
#pragma unroll
                    for (int m = 0; m < MT; ++m) {
                        if (P.zp.tok_zero && m < P.M) acc[m] -= P.zp.tok_zero[m] * rs;
                        usum[m] = fmaf((float)acc[m], h, usum[m]);
                        if (P.acc_out && m < P.M && n < P.L.N)
                            P.acc_out[((size_t)kb * P.M + m) * P.L.N + n] = acc[m];
                    }
                }
            }
        }
    }

    // partial sums of this slice, then find out whether every slice of the tile is in
    if (GROUPED) {
        float *part = reinterpret_cast<float *>(P.partials);
#pragma unroll
        for (int m = 0; m < MT; ++m)
            if (m < P.M) part[((size_t)slice * P.M + m) * P.L.n_pad + n] = usum[m];
    } else {
        int32_t *part = reinterpret_cast<int32_t *>(P.partials);
#pragma unroll
        for (int m = 0; m < MT; ++m)
            if (m < P.M) part[((size_t)slice * P.M + m) * P.L.n_pad + n] = acc[m];
    }
    __threadfence();
    __syncthreads();
    if (r == 0) {
        const int old = atomicAdd(P.counters + nt, 1);
        const int last = old == P.slices - 1;
        if (last) P.counters[nt] = 0;            // ready for the next call
        s_last = last;
    }
    __syncthreads();
    if (!s_last || n >= P.L.N) return;
    __threadfence();
    const float bias_n = P.bias ? P.bias[n] : 0.0f;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        if (m >= P.M) break;
        float tv;
        if (GROUPED) {
            const float *part = reinterpret_cast<const float *>(P.partials);
            float u = 0.0f;
#pragma unroll 8
            for (int s = 0; s < P.slices; ++s)               // loads of eight slices in flight
                u = __fadd_rn(u, __ldcg(part + ((size_t)s * P.M + m) * P.L.n_pad + n));
            tv = __fmul_rn(u, s_tok[m]);
        } else {
            const int32_t *part = reinterpret_cast<const int32_t *>(P.partials);
            int a = 0;
#pragma unroll 8
            for (int s = 0; s < P.slices; ++s)               // loads of eight slices in flight
                a += __ldcg(part + ((size_t)s * P.M + m) * P.L.n_pad + n);
            if (P.zp.tok_zero) a -= P.zp.tok_zero[m] * P.zp.rowsum[n];
            if (P.acc_out) P.acc_out[(size_t)m * P.L.N + n] = a;
            tv = rescale_channel(a, s_tok[m], __fmul_rn(P.unit, P.scales[n]));
        }
        if (P.bias) tv = __fadd_rn(tv, bias_n);
        if (P.Y) P.Y[(size_t)m * P.L.N + n] = __float2bfloat16_rn(tv);
    }
}

// ---------------------------------------------------------------------------
// Row-slab variant: one CTA owns 32 output rows over the whole of K.
// ---------------------------------------------------------------------------
// The K split happens inside the CTA (warp w takes k-blocks w, w + W, ...), the warps' sums meet
// in shared memory, and the CTA writes its 32 outputs itself: no partial sums in global memory,
// no atomic counter, no second phase.  For a weight stream of a few tens of megabytes that
// second phase and its round trips are a third of the launch.  A lane owns one row: per k-block
// it reads 4 x 16 bytes (a warp reads 4 x 512 contiguous bytes), two k-blocks ahead in registers.
constexpr int kRowsPerCta = 32;
constexpr int kRowSlabMaxTokenBytes = 96 * 1024;

// BITS = 3: the 3-bit tile layout (twelve 32-bit words per row and k-block, word w of all 128 rows
// contiguous, so a warp's 32 lanes read 128 contiguous bytes per word) and the 8-entry level
// table; no offset tables there (one permute per four codes already).
template <int MT, bool GROUPED, int W, int BITS = 4>
__global__ void __launch_bounds__(32 * W)
linear_gemv_rows_kernel(const GemvParams P)
{
    extern __shared__ __align__(16) uint8_t rows_smem[];
    int8_t *s_x = reinterpret_cast<int8_t *>(rows_smem);                       // [MT][K]
    int32_t *s_red = reinterpret_cast<int32_t *>(rows_smem + (size_t)MT * P.L.K);   // [W][MT][32]
    int *s_sum = s_red + W * MT * 32;     // [MT][k_blocks] sums of the tokens' values per k-block
    __shared__ float s_tok[MT];          // token steps (read or, in the fused form, computed here)
    allow_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nt = blockIdx.x >> 2, slab = blockIdx.x & 3;
    const int r = slab * kRowsPerCta + lane;                  // row inside the 128-row tile
    const int n = nt * kTileN + r;
    const int k_blocks = P.L.k_blocks;
    const uint8_t *src = BITS == 3 ? P.codes + (size_t)nt * k_blocks * kTileBytes3 + r * 4
                                   : P.codes + (size_t)nt * k_blocks * kTileBytes + r * 16;
    auto fetch = [&](int kb, uint4 (&dst)[4]) {
        if constexpr (BITS == 3) {
            uint32_t *d = reinterpret_cast<uint32_t *>(dst);        // twelve of the sixteen words
            const uint32_t *p = reinterpret_cast<const uint32_t *>(src + (size_t)kb * kTileBytes3);
#pragma unroll
            for (int i = 0; i < 12; ++i) {
                uint32_t v;
                asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p + i * 128));
                d[i] = v;
            }
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q)
                dst[q] = ld_stream(reinterpret_cast<const uint4 *>(src + (size_t)kb * kTileBytes +
                                                                   q * kQuarterBytes));
        }
    };
    // Before the wait only prefetch hints are allowed: ask L2 for this warp's first two
    // k-blocks (its 32 rows x 16 bytes x 4 quarters each = sixteen 128-byte lines per k-block, one
    // line per lane), so that their HBM round trip overlaps the tail of the kernel before.
    // (Hints further ahead inside the main loop were measured slower on the large shapes.)
    auto prefetch_pair = [&](int kb0) {      // k-blocks kb0 and kb0 + W of this warp
        const int kbp = kb0 + (lane >> 4) * W;
        if (BITS == 4 && kbp < k_blocks) {
            const uint8_t *line = P.codes + ((size_t)nt * k_blocks + kbp) * kTileBytes +
                                  ((lane >> 2) & 3) * kQuarterBytes + slab * (kRowsPerCta * 16) + (lane & 3) * 128;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(line));
        }
    };
    prefetch_pair(warp);
    // earlier work in the stream (the activation quantizer) is complete from here on
    dependent_wait();
    uint4 wa[4], wb[4];
    int kb = warp;
    if (kb < k_blocks) fetch(kb, wa);
    if (kb + W < k_blocks) fetch(kb + W, wb);
    // the tokens, whole rows, for all warps
    if (P.X) {
        // fused form: quantize the tokens here (the codes of the first k-blocks are on their way)
        float amax[MT];
        cta_token_absmax<MT>(P.X, P.inv_s, P.M, P.L.K, reinterpret_cast<float *>(s_red), amax);
        float rq[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            rq[m] = amax[m] > 0.0f ? __fdiv_rn(127.0f, amax[m]) : 0.0f;
            if (threadIdx.x == 0) s_tok[m] = amax[m] > 0.0f ? __fdiv_rn(amax[m], 127.0f) : 0.0f;
        }
        const int nvec = P.L.K / 8;
        for (int c = threadIdx.x; c < nvec; c += 32 * W) {
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                uint2 v = make_uint2(0u, 0u);
                if (m < P.M) v = quantize_vec8(P.X, P.inv_s, P.L.K, m, c, rq[m]);
                reinterpret_cast<uint2 *>(s_x + (size_t)m * P.L.K)[c] = v;
            }
        }
    } else {
        if (threadIdx.x < MT)
            s_tok[threadIdx.x] = (P.tok_scale && (int)threadIdx.x < P.M) ? P.tok_scale[threadIdx.x] : 0.0f;
        const int chunks = P.L.K / 16;
        for (int i = threadIdx.x; i < MT * chunks; i += 32 * W) {
            const int m = i / chunks, c = i - m * chunks;
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (m < P.M) v = __ldg(reinterpret_cast<const uint4 *>(P.Xq + (size_t)m * P.L.K) + c);
            reinterpret_cast<uint4 *>(s_x + (size_t)m * P.L.K)[c] = v;
        }
    }
    const bool blob_ok = header_matches(P.blob, P.L);
    __syncthreads();
    if (!blob_ok) {
        if (threadIdx.x == 0) report_failure(P.sb, W4A8_ERR_BAD_BLOB, 4);
        return;
    }
    // offset-table expansion (see build_offset_tables) for special values step/2 and step/4;
    // a warp sums the token values of its own k-blocks (written and read by the same warp)
    const bool offset_tables = BITS == 4 && P.L.shift <= 2;
    const int off = 13 << P.L.shift;
    if (offset_tables) {
        for (int kbi = warp; kbi < k_blocks; kbi += W)
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                const int sum = warp_sum128(s_x + (size_t)m * P.L.K + kbi * kTileK);
                if (lane == 0) s_sum[m * k_blocks + kbi] = sum;
            }
        __syncwarp();
    }
    int acc[MT];
    float usum[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) { acc[m] = 0; usum[m] = 0.0f; }
    uint32_t t[4];
    auto tables = [&](int z) {
        if constexpr (BITS == 3) {
            uint32_t t3[2];
            build_level_tables3(z, P.L.shift, t3);
            t[0] = t3[0]; t[1] = t3[1];
        } else {
            if (offset_tables) build_offset_tables(z, P.lt, P.L.shift, t);
            else build_level_tables(z, P.lt, t);
        }
    };
    if (!GROUPED) tables(P.zeros[n]);
    auto consume = [&](int kbi, const uint4 (&w)[4]) {
        if (GROUPED) {
            tables(P.zeros[(size_t)kbi * P.L.n_pad + n]);
#pragma unroll
            for (int m = 0; m < MT; ++m) acc[m] = 0;
        }
        if constexpr (BITS == 3) {
            // per 32-k quarter: three words whose nibbles (top bit cleared) select eight levels
            // each, and a fourth selector put together from the top bits
            const uint32_t *w3 = reinterpret_cast<const uint32_t *>(w);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t a = w3[3 * q], b = w3[3 * q + 1], c = w3[3 * q + 2];
                const uint32_t sel[4] = {a & 0x77777777u, b & 0x77777777u, c & 0x77777777u,
                                         ((a >> 3) & 0x11111111u) | ((b >> 2) & 0x22222222u) |
                                             ((c >> 1) & 0x44444444u)};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t d0 = prmt(t[0], t[1], sel[j]), d1 = prmt(t[0], t[1], sel[j] >> 16);
#pragma unroll
                    for (int m = 0; m < MT; ++m) {
                        const uint2 x = *reinterpret_cast<const uint2 *>(
                            s_x + (size_t)m * P.L.K + kbi * kTileK + q * 32 + j * 8);
                        acc[m] = __dp4a((int)d0, (int)x.x, acc[m]);
                        acc[m] = __dp4a((int)d1, (int)x.y, acc[m]);
                    }
                }
            }
        } else if (offset_tables) {
            block_dot_offset<MT>(w, t, s_x + kbi * kTileK, (size_t)P.L.K, acc);
#pragma unroll
            for (int m = 0; m < MT; ++m)
                acc[m] = (int)((uint32_t)acc[m] - (uint32_t)off * (uint32_t)s_sum[m * k_blocks + kbi]);
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t words[4] = {w[q].x, w[q].y, w[q].z, w[q].w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint32_t d0, d1;
                    decode8(words[i], t, d0, d1);
#pragma unroll
                    for (int m = 0; m < MT; ++m) {
                        const uint2 x = *reinterpret_cast<const uint2 *>(
                            s_x + (size_t)m * P.L.K + kbi * kTileK + q * 32 + i * 8);
                        acc[m] = __dp4a((int)d0, (int)x.x, acc[m]);
                        acc[m] = __dp4a((int)d1, (int)x.y, acc[m]);
                    }
                }
            }
        }
        if (GROUPED) {
            const float h = __fmul_rn(P.unit, P.scales[(size_t)kbi * P.L.n_pad + n]);
            const int rs = (P.zp.tok_zero && n < P.L.N) ? P.zp.rowsum[(size_t)kbi * P.L.N + n] : 0;
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                if (P.zp.tok_zero && m < P.M) acc[m] -= P.zp.tok_zero[m] * rs;
                usum[m] = fmaf((float)acc[m], h, usum[m]);
                if (P.acc_out && m < P.M && n < P.L.N)
                    P.acc_out[((size_t)kbi * P.M + m) * P.L.N + n] = acc[m];
            }
        }
    };
    // two register sets alternate; each is refilled right after it has been consumed
    for (; kb < k_blocks; kb += 2 * W) {
        consume(kb, wa);
        if (kb + 2 * W < k_blocks) fetch(kb + 2 * W, wa);
        if (kb + W < k_blocks) {
            consume(kb + W, wb);
            if (kb + 3 * W < k_blocks) fetch(kb + 3 * W, wb);
        }
    }
#pragma unroll
    for (int m = 0; m < MT; ++m)
        s_red[(warp * MT + m) * 32 + lane] = GROUPED ? (int32_t)__float_as_int(usum[m]) : acc[m];
    __syncthreads();
    if (warp != 0 || n >= P.L.N) return;
    const float bias_n = P.bias ? P.bias[n] : 0.0f;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        if (m >= P.M) break;
        float tv;
        if (GROUPED) {
            float u = 0.0f;
            for (int w = 0; w < W; ++w) u = __fadd_rn(u, __int_as_float(s_red[(w * MT + m) * 32 + lane]));
            tv = __fmul_rn(u, s_tok[m]);
        } else {
            int a = 0;
            for (int w = 0; w < W; ++w) a += s_red[(w * MT + m) * 32 + lane];
            if (P.zp.tok_zero) a -= P.zp.tok_zero[m] * P.zp.rowsum[n];
            if (P.acc_out) P.acc_out[(size_t)m * P.L.N + n] = a;
            tv = rescale_channel(a, s_tok[m], __fmul_rn(P.unit, P.scales[n]));
        }
        if (P.bias) tv = __fadd_rn(tv, bias_n);
        if (P.Y) P.Y[(size_t)m * P.L.N + n] = __float2bfloat16_rn(tv);
    }
}

// Raise a kernel's dynamic shared-memory limit to `bytes` unless an earlier call on this device
// already set it at least that high (one slot per kernel instance and device).
template <typename Kernel>
void ensure_dynamic_smem(Kernel kern, int bytes, std::atomic<int> (&set_bytes)[kMaxGemvDevices])
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxGemvDevices) dev = -1;
    if (dev >= 0 && set_bytes[dev].load(std::memory_order_acquire) >= bytes) return;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess &&
        dev >= 0)
        set_bytes[dev].store(bytes, std::memory_order_release);
}

template <int MT, bool GROUPED, int W, int BITS = 4>
void launch_rows(const GemvParams &P, cudaStream_t st)
{
    const int smem = MT * P.L.K + W * MT * 32 * 4 + MT * P.L.k_blocks * 4;
    static std::atomic<int> set_bytes[kMaxGemvDevices] = {};
    ensure_dynamic_smem(linear_gemv_rows_kernel<MT, GROUPED, W, BITS>, smem, set_bytes);
    launch_overlapped(linear_gemv_rows_kernel<MT, GROUPED, W, BITS>, dim3(P.L.n_tiles * 4), dim3(32 * W),
                      (size_t)smem, st, P);
}

// As many warps per row-slab CTA as keep the whole grid resident at once (32 warps of 64
// registers per SM on every SM): a second wave of CTAs repeats the start-up latency.  Measured on
// 4096 -> 16384: 13.9 us with 16 warps (1.7 waves), 11.6 us with 8 (all resident).
inline int resident_warps() { return device_sms() * 32; }
inline int row_slab_warps(int mt, const BlobLayout &L)
{
    const int slabs = L.n_tiles * 4;
    const int kResidentWarps = resident_warps();
    if (mt <= 2 && slabs * 32 <= kResidentWarps && L.k_blocks >= 32) return 32;
    if (slabs * 16 <= kResidentWarps && L.k_blocks >= 32) return 16;
    if (slabs * 8 <= kResidentWarps && L.k_blocks >= 16) return 8;
    return L.k_blocks >= 64 ? 8 : 4;
}

template <int MT, bool GROUPED>
void launch_rows_w(const GemvParams &P, cudaStream_t st, int warps)
{
    if (warps == 0) warps = row_slab_warps(MT, P.L);
    if (warps == 32) {
        // 1024 threads leave 64 registers each: enough for one or two tokens only
        if constexpr (MT <= 2) launch_rows<MT, GROUPED, 32>(P, st);
        else launch_rows<MT, GROUPED, 16>(P, st);
    } else if (warps == 16) launch_rows<MT, GROUPED, 16>(P, st);
    else if (warps == 8) launch_rows<MT, GROUPED, 8>(P, st);
    else launch_rows<MT, GROUPED, 4>(P, st);
}

// enough row slabs to occupy the GPU, and the tokens fit in shared memory
inline bool row_slabs_fit(int M, const BlobLayout &L, bool requested)
{
    const int mt = M == 1 ? 1 : (M == 2 ? 2 : 4);
    const int slabs = L.n_tiles * 4;
    if ((size_t)mt * L.K > (size_t)kRowSlabMaxTokenBytes) return false;
    if (requested) return true;              // the caller named the warps of a row-slab CTA
    // Fewer slabs than SMs and a long K: with four tokens a CTA has at most 16 warps and would
    // stream too much alone (the K-sliced kernel is faster there); with one or two tokens a CTA
    // of 32 warps keeps enough in flight (16384 -> 4096, one token: 11.6 us against 15.0 us).
    if (mt > 2 && slabs < device_sms() && L.k_blocks > 96) return false;
    return slabs >= 96;
}

template <int MT, bool GROUPED>
void launch_gemv(dim3 grid, const GemvParams &P, cudaStream_t st)
{
    constexpr int smem = kGemvRingBytes + MT * kGemvMaxSteps * kGemvKb * kTileK;
    static std::atomic<int> set_bytes[kMaxGemvDevices] = {};
    ensure_dynamic_smem(linear_gemv_kernel<MT, GROUPED>, smem, set_bytes);
    launch_overlapped(linear_gemv_kernel<MT, GROUPED>, grid, dim3(128), smem, st, P);
}

}  // namespace

int gemv_max_tokens() { return kGemvMaxTokens; }

int gemv_row_slab_warps(int M, const BlobLayout &L, int requested_warps)
{
    if (!row_slabs_fit(M, L, requested_warps != 0)) return 0;
    const int mt = M == 1 ? 1 : (M == 2 ? 2 : 4);
    int w = requested_warps ? requested_warps : row_slab_warps(mt, L);
    if (w == 32 && mt > 2) w = 16;
    if (L.bits == 3) {                 // 3-bit codes: one or two tokens, 8 or 16 warps
        if (M > 2) return 0;
        w = w >= 16 ? 16 : 8;
    }
    return w;
}

// Whether the one-launch decode form should quantize the tokens inside the weight-streaming
// kernel: yes while the grid is resident at once (every CTA repeats the quantizer once); on a
// matrix whose row slabs come in several waves each wave would repeat it, and a quantizer launch
// of its own in front is faster (9216 -> 36864, one token: 35 against 38 us).
bool gemv_quantize_inside(int M, const BlobLayout &L)
{
    if (!row_slabs_fit(M, L, false)) return true;        // the K-sliced grid is sized to be resident
    const int mt = M == 1 ? 1 : (M == 2 ? 2 : 4);
    return L.n_tiles * 4 * row_slab_warps(mt, L) <= resident_warps();
}

// Workspace of the GEMV path: status block, one counter per row tile, partial sums
// [slices][M][n_pad] (4 bytes each).
void gemv_plan(int M, const BlobLayout &L, LinearPlan *plan)
{
    // K slices so that the grid fills, but does not exceed, six CTAs per SM when it can;
    // a slice is between 2 and 16 k-blocks
    const int target_ctas = device_sms() * 6;
    int slices = target_ctas / L.n_tiles;
    if (slices < 1) slices = 1;
    int per = (L.k_blocks + slices - 1) / slices;
    if (per < kGemvKb) per = kGemvKb;
    if (per > kGemvKb * kGemvMaxSteps) per = kGemvKb * kGemvMaxSteps;
    if (per > L.k_blocks) per = L.k_blocks;
    slices = (L.k_blocks + per - 1) / per;
    plan->tok_tile = 0;
    plan->tok_tiles = 1;
    plan->split_k = slices;
    plan->kb_per_split = per;
    plan->decode_warps = 0;
    plan->off_counters = sizeof(StatusBlock);
    plan->off_partials = align_up(plan->off_counters + (size_t)L.n_tiles * sizeof(int), 256);
    plan->workspace_bytes = plan->off_partials + (size_t)slices * M * L.n_pad * 4;
}

w4a8_status launch_linear_gemv(const int8_t *Xq, const float *tok_scale, const uint8_t *blob,
                               const BlobLayout &L, const float *bias, int M, __nv_bfloat16 *Y,
                               int32_t *acc, uint8_t *workspace, const LinearPlan &plan,
                               cudaStream_t st, ZeroPoint zp, const __half *X, const float *inv_s)
{
    if (M < 1 || M > kGemvMaxTokens) return W4A8_ERR_SHAPE;
    GemvParams P;
    P.X = X;
    P.inv_s = inv_s;
    P.blob = blob;
    P.codes = blob + L.off_codes;
    P.scales = reinterpret_cast<const float *>(blob + L.off_scales);
    P.zeros = blob + L.off_zeros;
    P.Xq = Xq;
    P.tok_scale = tok_scale;
    P.bias = bias;
    P.Y = Y;
    P.acc_out = acc;
    P.sb = reinterpret_cast<StatusBlock *>(workspace);
    P.counters = reinterpret_cast<int *>(workspace + plan.off_counters);
    P.partials = workspace + plan.off_partials;
    P.L = L;
    P.M = M;
    P.slices = plan.split_k;
    P.kb_per_slice = plan.kb_per_split;
    P.zp = zp;
    P.lt = make_level_tables(L.shift);
    P.unit = level_unit(L.shift);
    if (P.slices > 65535) return W4A8_ERR_SHAPE;
    const dim3 grid(L.n_tiles, P.slices);
    const bool g = L.group != 0;
    if (L.bits == 3) {
        // 3-bit codes: the row-slab kernel only, one or two tokens, 8 or 16 warps per CTA
        if (M > 2 || X != nullptr || !row_slabs_fit(M, L, plan.decode_warps != 0)) return W4A8_ERR_SHAPE;
        int w = plan.decode_warps ? plan.decode_warps : row_slab_warps(M, L);
        w = w >= 16 ? 16 : 8;
        if (M == 1) {
            if (g) { if (w == 16) launch_rows<1, true, 16, 3>(P, st); else launch_rows<1, true, 8, 3>(P, st); }
            else { if (w == 16) launch_rows<1, false, 16, 3>(P, st); else launch_rows<1, false, 8, 3>(P, st); }
        } else {
            if (g) { if (w == 16) launch_rows<2, true, 16, 3>(P, st); else launch_rows<2, true, 8, 3>(P, st); }
            else { if (w == 16) launch_rows<2, false, 16, 3>(P, st); else launch_rows<2, false, 8, 3>(P, st); }
        }
        return cudaGetLastError() == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
    }
    if (row_slabs_fit(M, L, plan.decode_warps != 0)) {
        const int w = plan.decode_warps;
        if (M == 1) { if (g) launch_rows_w<1, true>(P, st, w); else launch_rows_w<1, false>(P, st, w); }
        else if (M == 2) { if (g) launch_rows_w<2, true>(P, st, w); else launch_rows_w<2, false>(P, st, w); }
        else { if (g) launch_rows_w<4, true>(P, st, w); else launch_rows_w<4, false>(P, st, w); }
        return cudaGetLastError() == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
    }
    if (M == 1) {
        if (g) launch_gemv<1, true>(grid, P, st);
        else launch_gemv<1, false>(grid, P, st);
    } else if (M == 2) {
        if (g) launch_gemv<2, true>(grid, P, st);
        else launch_gemv<2, false>(grid, P, st);
    } else {
        if (g) launch_gemv<4, true>(grid, P, st);
        else launch_gemv<4, false>(grid, P, st);
    }
    return cudaGetLastError() == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

}  // namespace w4a8
