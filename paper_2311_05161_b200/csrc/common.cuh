// Shared declarations of the W4A8-dINT CUDA library: blob layout, status block,
// exact-arithmetic helpers.  sm_100a only.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "w4a8.h"

namespace w4a8 {

// ---------------------------------------------------------------------------
// packed-weight blob
// ---------------------------------------------------------------------------
constexpr int kTileN = 128;        // output rows per code tile
constexpr int kTileK = 128;        // input features per code tile (= one quantization group)
constexpr int kTileBytes = 8192;   // 128 x 128 nibbles (4-bit codes)
constexpr int kQuarterBytes = 2048;
// 3-bit codes (dINT3): a tile is 128 x 128 x 3 bits.  Per 32-k quarter and row three 32-bit
// words hold 32 codes: nibble j of word w (w = 0, 1, 2) carries in its low three bits the code
// of k = 8 w + j, and the three spare top bits of the nibbles j of words 0, 1, 2 are bits 0,
// 1, 2 of the code of k = 24 + j.  Word w of row r of quarter q sits at byte
// q * 1536 + w * 512 + r * 4, so a warp reads 128 contiguous bytes per word.
constexpr int kTileBytes3 = 6144;
constexpr int kQuarterBytes3 = 1536;
constexpr int kHeaderBytes = 256;
constexpr uint32_t kBlobMagic = 0x38413457u;   // "W4A8"
constexpr uint32_t kBlobVersion = 1u;
constexpr uint32_t kBlobLayoutQuarterRow16 = 1u;

struct BlobHeader {
    uint32_t magic, version, layout, group;
    int32_t N, K, G, n_tiles, k_blocks, n_pad;
    uint32_t level_shift;   // special value = step / 2^level_shift; 0 (older blobs) means 1
    uint32_t bits;          // code width: 3 or 4; 0 (older blobs) means 4
    uint64_t off_scales, off_zeros, off_codes, total_bytes;
    float clip;
    uint32_t pad1[43];
};
static_assert(sizeof(BlobHeader) == kHeaderBytes, "blob header is 256 bytes");

struct BlobLayout {
    int N, K, group, G, n_tiles, k_blocks, n_pad;
    int shift;              // special value = step / 2^shift (1, 2 or 3); levels are in that unit
    int bits;               // code width b: 4 (p = 13 integer steps) or 3 (p = 5)
    int tile_bytes;         // bytes of one 128 x 128 code tile: 8192 or 6144
    size_t off_scales, off_zeros, off_codes, total_bytes;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__host__ __device__ inline BlobLayout make_layout(int N, int K, int group, int shift = 1,
                                                  int bits = 4)
{
    BlobLayout L;
    L.shift = shift;
    L.bits = bits;
    L.tile_bytes = bits == 3 ? kTileBytes3 : kTileBytes;
    L.N = N;
    L.K = K;
    L.group = group;
    L.G = group ? K / group : 1;
    L.n_tiles = (N + kTileN - 1) / kTileN;
    L.k_blocks = K / kTileK;
    L.n_pad = L.n_tiles * kTileN;
    L.off_scales = kHeaderBytes;
    L.off_zeros = align_up(L.off_scales + (size_t)L.G * L.n_pad * sizeof(float), 256);
    L.off_codes = align_up(L.off_zeros + (size_t)L.G * L.n_pad, 256);
    L.total_bytes = L.off_codes + (size_t)L.n_tiles * L.k_blocks * L.tile_bytes;
    return L;
}

// Byte offset, inside the code section, of the byte holding code[n][k] (k even: low nibble).
__host__ __device__ inline size_t code_byte_offset(const BlobLayout &L, int n, int k)
{
    const int nt = n / kTileN, r = n % kTileN;
    const int kb = k / kTileK, kk = k % kTileK;
    const int q = kk / 32, j = (kk % 32) / 2;
    return ((size_t)nt * L.k_blocks + kb) * kTileBytes + (size_t)q * kQuarterBytes + r * 16 + j;
}

inline bool bits_ok(int bits) { return bits == 3 || bits == 4; }

inline bool shape_ok(int N, int K, int group)
{
    if (N < 8 || N % 8 != 0) return false;
    if (K < 128 || K % 128 != 0 || K >= (1 << 19)) return false;
    if (group != 0 && group != 128) return false;
    return true;
}

__device__ inline bool header_matches(const uint8_t *blob, const BlobLayout &L)
{
    const BlobHeader *h = reinterpret_cast<const BlobHeader *>(blob);
    return h->magic == kBlobMagic && h->version == kBlobVersion &&
           h->layout == kBlobLayoutQuarterRow16 && h->N == L.N && h->K == L.K &&
           h->group == (uint32_t)L.group &&
           (h->level_shift == 0u ? 1u : h->level_shift) == (uint32_t)L.shift &&
           (h->bits == 0u ? 4u : h->bits) == (uint32_t)L.bits;
}

// The 3-bit code of k = 32 q + i of a row from the row's three words of quarter q.
__host__ __device__ inline int code3_of(uint32_t w0, uint32_t w1, uint32_t w2, int i)
{
    if (i < 24) {
        const uint32_t w = i < 8 ? w0 : (i < 16 ? w1 : w2);
        return (int)((w >> (4 * (i & 7))) & 7u);
    }
    const int sh = 4 * (i - 24) + 3;
    return (int)(((w0 >> sh) & 1u) | (((w1 >> sh) & 1u) << 1) | (((w2 >> sh) & 1u) << 2));
}
// Byte offset, inside the code section, of word w of the 3-bit codes of row n, quarter (kb, q).
__host__ __device__ inline size_t code3_word_offset(const BlobLayout &L, int n, int kb, int q, int w)
{
    const int nt = n / kTileN, r = n % kTileN;
    return ((size_t)nt * L.k_blocks + kb) * kTileBytes3 + (size_t)q * kQuarterBytes3 + w * 512 + r * 4;
}

// ---------------------------------------------------------------------------
// status block (first 256 bytes of a workspace)
// ---------------------------------------------------------------------------
struct StatusBlock {
    int status;       // 0, W4A8_ERR_TIMEOUT or W4A8_ERR_BAD_BLOB: first failure wins
    int where;        // site code of the wait that gave up
    int block;        // CTA that reported
    int pad[61];
};
static_assert(sizeof(StatusBlock) == 256, "status block is 256 bytes");

__device__ inline void report_failure(StatusBlock *sb, int status, int where)
{
    if (atomicCAS(&sb->status, 0, status) == 0) {
        sb->where = where;
        sb->block = (int)blockIdx.x;
    }
}

// ---------------------------------------------------------------------------
// dINT4 decode (Eq. 6) in units of the special value c = step / 2^shift, so that every
// level is an integer: 2^shift (code - z) for the integer levels, +1 for c1, -1 for c2.
// shift = 1 is the paper's c = step / 2; App. A.5 also tries step / 4 and step / 8.
// ---------------------------------------------------------------------------
__host__ __device__ inline int dint4_level(int code, int z, int shift)
{
    return code <= 13 ? (code - z) * (1 << shift) : (code == 14 ? 1 : -1);
}
// the same for b-bit codes: integer codes 0..p, p + 1 = +c, p + 2 = -c, p = 2^b - 3
__host__ __device__ inline int dint_level(int code, int z, int shift, int bits)
{
    const int p = (1 << bits) - 3;
    return code <= p ? (code - z) * (1 << shift) : (code == p + 1 ? 1 : -1);
}
// the unit itself as a factor of the step: 2^-shift, exact
__host__ __device__ inline float level_unit(int shift)
{
    return shift == 1 ? 0.5f : (shift == 2 ? 0.25f : 0.125f);
}
// Byte tables of the levels for the permute-based decode: table word w, byte i holds the level
// of code 4 w + i.  A thread builds them as (base[w] - z * zmul) ^ 0x80808080 (bytes carry a
// 0x80 offset so that the subtraction never borrows); base and zmul depend on the shift only.
struct LevelTables {
    uint32_t base[4];
    uint32_t zmul;
};
inline LevelTables make_level_tables(int shift)
{
    const uint32_t m = 1u << shift;
    LevelTables t;
    t.base[0] = 0x80808080u + m * 0x03020100u;
    t.base[1] = 0x80808080u + m * 0x07060504u;
    t.base[2] = 0x80808080u + m * 0x0B0A0908u;
    t.base[3] = 0x00008080u + m * 0x00000D0Cu;
    t.zmul = m * 0x01010101u;
    return t;
}
// 3-bit codes: eight levels in two words (codes 0..3, then 4, 5, +1, -1).
__device__ __forceinline__ void build_level_tables3(int z, int shift, uint32_t (&t)[2])
{
    const uint32_t m = 1u << shift;
    const uint32_t zz = (uint32_t)z * m * 0x01010101u;
    t[0] = ((0x80808080u + m * 0x03020100u) - zz) ^ 0x80808080u;
    t[1] = ((((0x00008080u + m * 0x00000504u) - (zz & 0xFFFFu)) ^ 0x00008080u) & 0xFFFFu) | 0xFF010000u;
}
__device__ __forceinline__ void build_level_tables(int z, const LevelTables &lt, uint32_t (&t)[4])
{
    const uint32_t zz = (uint32_t)z * lt.zmul;
    t[0] = (lt.base[0] - zz) ^ 0x80808080u;
    t[1] = (lt.base[1] - zz) ^ 0x80808080u;
    t[2] = (lt.base[2] - zz) ^ 0x80808080u;
    // codes 12 and 13, then the two special values +1 and -1
    t[3] = (((lt.base[3] - (zz & 0xFFFFu)) ^ 0x00008080u) & 0xFFFFu) | 0xFF010000u;
}

// ---------------------------------------------------------------------------
// output rescale, one rounded FP32 operation per step
// ---------------------------------------------------------------------------
__device__ inline float rescale_channel(int acc, float tok_scale, float half_step)
{
    return __fmul_rn(__fmul_rn((float)acc, tok_scale), half_step);
}

__device__ inline float add_bias(float t, const float *bias, int n)
{
    return bias ? __fadd_rn(t, bias[n]) : t;
}

// ---------------------------------------------------------------------------
// ---------------------------------------------------------------------------
// programmatic dependent launch
// ---------------------------------------------------------------------------
// The hot kernels (activation quantizer, both linear kernels) are launched so that one may
// start while the kernel before it in the stream is still draining: launch latency, CTA
// scheduling and each kernel's set-up then overlap the predecessor's tail.  The rule every
// such kernel keeps: before dependent_wait() it touches no global memory except prefetch
// hints; dependent_wait() returns once all earlier work in the stream is complete and visible.
// Kernels launched the ordinary way (packing, the reference kernel) order as always.
__device__ __forceinline__ void allow_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void dependent_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

#ifdef __CUDACC__
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block,
                                             size_t smem, cudaStream_t st, int cluster,
                                             Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = 1;
    if (cluster > 1) {                  // thread-block clusters of `cluster` CTAs along x
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)cluster;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    cfg.attrs = attr;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                     cudaStream_t st, Args &&...args)
{
    return launch_overlapped_cluster(kernel, grid, block, smem, st, 1, static_cast<Args &&>(args)...);
}
#endif

// plan of the tensor-core kernel (shared by the workspace query and the launcher)
// ---------------------------------------------------------------------------
struct LinearPlan {
    int tok_tile;     // tokens per tile (UMMA N): 16, 32, 64, 128, 256
    int tok_tiles;    // ceil(M / tok_tile)
    int split_k;      // K slices (1 = none)
    int decode_warps; // warps converting codes to INT8: 4, 8 or 16
    int cluster;      // CTAs per cluster: 1, or 2 (each CTA expands half of every code tile for both)
    int debug_wait_ms, debug_skip_load;   // test hooks of w4a8_opts (0 = off)
    int swiglu;       // gated-unit epilogue (see w4a8_linear_swiglu)
    int tok_run;      // token tiles per run of the unit order on request, 0 = automatic
    int batched;      // every 128-row tile has its own block of tokens (attention P*V form)
    int kb_per_split; // k-blocks per slice (last slice may be shorter)
    int offset;       // 0, or the offset of the decode tables (13 * 2^shift)
    size_t toksum_slots;
    size_t off_counters, off_partials, off_toksum, workspace_bytes;
};

// Asymmetric activations: acc[m][n] -= tok_zero[m] * rowsum[n] before the rescale (both
// pointers NULL for the symmetric path).
struct ZeroPoint {
    const int32_t *tok_zero = nullptr;   // [M]
    const int32_t *rowsum = nullptr;     // [N]
};

// SM count of the current device (asked on every call: a process may drive several devices;
// 148, a B200, when no device answers, so that the size queries work without one)
int device_sms();
// L2 size of the current device in bytes
long long device_l2_bytes();

// launchers (defined in the .cu files, called by api.cu)
cudaError_t launch_pack(const __half *W, const float *s_in, const BlobLayout &L, float clip,
                        uint8_t *blob, cudaStream_t st);
cudaError_t launch_pack_transposed(const __half *Wt, const BlobLayout &L, float clip, uint8_t *blob,
                                   cudaStream_t st);
cudaError_t launch_unpack(const uint8_t *blob, const BlobLayout &L, uint8_t *codes,
                          float *scales, uint8_t *zeros, cudaStream_t st);
cudaError_t launch_quantize_act(const __half *X, const float *inv_s, int M, int K, int8_t *Xq,
                                float *tok_scale, cudaStream_t st);
cudaError_t launch_quantize_act_asym(const __half *X, const float *inv_s, int M, int K, int8_t *Xq,
                                     float *tok_scale, int32_t *tok_zero, cudaStream_t st);
cudaError_t launch_norm_quantize_act(const __half *X, const float *weight, const float *bias,
                                     int layer_norm, float eps, int M, int K, int8_t *Xq,
                                     float *tok_scale, cudaStream_t st);
cudaError_t launch_weight_rowsum(const uint8_t *blob, const BlobLayout &L, int32_t *rowsum,
                                 cudaStream_t st);
cudaError_t launch_linear_simple(const int8_t *Xq, const float *tok_scale, const uint8_t *blob,
                                 const BlobLayout &L, const float *bias, int M,
                                 __nv_bfloat16 *Y, int32_t *acc, StatusBlock *sb,
                                 cudaStream_t st, ZeroPoint zp = ZeroPoint());
// auto_pair: the automatic plan may choose the MMA pair with offset tables (callers whose token
// layout or epilogue the pair does not cover leave it off)
bool make_plan(int M, const BlobLayout &L, const w4a8_opts *opts, LinearPlan *plan, bool auto_pair = false);
w4a8_status launch_linear_tcgen05(const int8_t *Xq, const float *tok_scale, const uint8_t *blob,
                                  const BlobLayout &L, const float *bias, int M,
                                  __nv_bfloat16 *Y, int32_t *acc, uint8_t *workspace,
                                  const LinearPlan &plan, cudaStream_t st,
                                  ZeroPoint zp = ZeroPoint());

int gemv_max_tokens();
bool gemv_quantize_inside(int M, const BlobLayout &L);
// warps of a row-slab CTA for this shape, 0 when the K-sliced variant runs instead
int gemv_row_slab_warps(int M, const BlobLayout &L, int requested_warps);
void gemv_plan(int M, const BlobLayout &L, LinearPlan *plan);
w4a8_status launch_linear_gemv(const int8_t *Xq, const float *tok_scale, const uint8_t *blob,
                               const BlobLayout &L, const float *bias, int M, __nv_bfloat16 *Y,
                               int32_t *acc, uint8_t *workspace, const LinearPlan &plan,
                               cudaStream_t st, ZeroPoint zp = ZeroPoint(),
                               const __half *X = nullptr, const float *inv_s = nullptr);

}  // namespace w4a8
