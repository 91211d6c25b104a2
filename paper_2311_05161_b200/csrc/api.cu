// extern "C" entry points: argument validation and dispatch.  See include/w4a8.h.
#include "common.cuh"

using namespace w4a8;

namespace w4a8 {

int device_sms()
{
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
        return v;
    cudaGetLastError();          // no device: not an error for the host-only queries
    return 148;
}

long long device_l2_bytes()
{
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&v, cudaDevAttrL2CacheSize, dev) == cudaSuccess && v > 0)
        return v;
    cudaGetLastError();
    return 126ll << 20;
}

}  // namespace w4a8

namespace {

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// W4A8_OK when the current device is compute capability 10.x.
w4a8_status check_arch()
{
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return W4A8_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return W4A8_ERR_CUDA;
    return major == 10 ? W4A8_OK : W4A8_ERR_UNSUPPORTED_ARCH;
}

bool opts_ok(const w4a8_opts *o)
{
    if (!o) return true;
    if (o->path < W4A8_PATH_AUTO || o->path > W4A8_PATH_GEMV) return false;
    if (o->split_k < 0 || o->tok_tile < 0 || o->decode_warps < 0) return false;
    if (o->level_shift < 0 || o->level_shift > 3) return false;
    if (o->cluster < 0 || o->cluster > 5) return false;
    if (o->tok_run < 0 || (o->tok_run && (o->path == W4A8_PATH_GEMV || o->path == W4A8_PATH_SIMPLE))) return false;
    if (o->offset_tables < 0 || o->offset_tables > 1 || (o->bits != 0 && !bits_ok(o->bits))) return false;
    if (o->offset_tables && (o->path == W4A8_PATH_GEMV || o->path == W4A8_PATH_SIMPLE)) return false;
    if (o->bits == 3 && o->cluster >= 2) return false;
#ifdef W4A8_DEBUG_HOOKS
    if (o->debug_wait_ms < 0 || o->debug_wait_ms > 2000 || o->debug_skip_load < 0) return false;
    if ((o->debug_wait_ms || o->debug_skip_load) && o->path != W4A8_PATH_TCGEN05) return false;
#else
    if (o->debug_wait_ms != 0 || o->debug_skip_load != 0) return false;
#endif
    return true;
}

// special value = step / 2^shift; 0 in the options means the paper's 1
int shift_of(const w4a8_opts *o) { return (o && o->level_shift) ? o->level_shift : 1; }
int bits_of(const w4a8_opts *o) { return (o && o->bits) ? o->bits : 4; }

// |level| <= 13 * 2^shift and |activation| <= amax: the INT32 sums must not overflow
bool depth_ok(int K, int shift, int amax)
{
    return (long long)K * amax * (13LL << shift) < (1LL << 31);
}

// The weight-streaming kernel can serve one to four tokens (on request, any of them).  By
// default it takes one and two tokens: measured, it is as fast or faster there on every shape
// (two tokens: 5.0 against 9.3 us on 4096 -> 4096, 13.2 against 17.7 us on 16384 -> 4096, equal on
// 9216 -> 36864), and the tensor-core kernel with its 16-token tile wins from four tokens on.
bool use_gemv(int M, const BlobLayout &L, const w4a8_opts *o)
{
    const int path = o ? o->path : W4A8_PATH_AUTO;
    if (path == W4A8_PATH_GEMV) return true;
    if (path != W4A8_PATH_AUTO || (o && (o->split_k || o->tok_tile || o->decode_warps || o->cluster || o->offset_tables || o->tok_run)))
        return false;
    // 3-bit tiles are read by the row-slab kernel only: layers too narrow for it stay on the
    // tensor-core kernel
    if (L.bits == 3) return M <= 2 && gemv_row_slab_warps(M, L, 0) > 0;
    return M <= 2;
}

w4a8_status linear_common(const int8_t *Xq, const float *tok_scale, const void *packed,
                          const float *bias, int M, int N, int K, int group, void *Y,
                          int32_t *acc, void *workspace, size_t workspace_bytes, void *stream,
                          const w4a8_opts *opts, ZeroPoint zp = ZeroPoint())
{
    if (!Xq || !packed || !workspace) return W4A8_ERR_NULL;
    if (!Y && !acc) return W4A8_ERR_NULL;
    if (Y && !tok_scale) return W4A8_ERR_NULL;
    if (!shape_ok(N, K, group) || M < 1 || !opts_ok(opts)) return W4A8_ERR_SHAPE;
    if (!depth_ok(K, shift_of(opts), zp.tok_zero ? 255 : 127)) return W4A8_ERR_SHAPE;
    if (!aligned(Xq, 16) || !aligned(tok_scale, 4) || !aligned(bias, 4) || !aligned(Y, 16) ||
        !aligned(acc, 16) || !aligned(packed, 256) || !aligned(workspace, 256))
        return W4A8_ERR_ALIGN;
    const size_t need = w4a8_linear_workspace_bytes_ex(M, N, K, group, opts);
    if (need == 0) return W4A8_ERR_SHAPE;
    if (workspace_bytes < need) return W4A8_ERR_BUFFER_TOO_SMALL;
    const w4a8_status arch = check_arch();
    if (arch != W4A8_OK) return arch;
    const BlobLayout L = make_layout(N, K, group, shift_of(opts), bits_of(opts));
    if (L.bits == 3 && zp.tok_zero) return W4A8_ERR_SHAPE;      // no row sums for 3-bit tiles
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint8_t *blob = static_cast<const uint8_t *>(packed);
    if (opts && opts->path == W4A8_PATH_SIMPLE) {
        const cudaError_t e =
            launch_linear_simple(Xq, tok_scale, blob, L, bias, M, static_cast<__nv_bfloat16 *>(Y),
                                 acc, static_cast<StatusBlock *>(workspace), st, zp);
        if (e == cudaErrorInvalidValue) return W4A8_ERR_SHAPE;
        return e == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
    }
    LinearPlan plan;
    if (use_gemv(M, L, opts)) {
        gemv_plan(M, L, &plan);
        // on request, the warps of a CTA of the row-slab variant (else chosen by the length of K)
        const int dw = opts ? opts->decode_warps : 0;
        if (dw != 0 && dw != 4 && dw != 8 && dw != 16 && dw != 32) return W4A8_ERR_SHAPE;
        plan.decode_warps = dw;
        return launch_linear_gemv(Xq, tok_scale, blob, L, bias, M, static_cast<__nv_bfloat16 *>(Y),
                                  acc, static_cast<uint8_t *>(workspace), plan, st, zp);
    }
    if (!make_plan(M, L, opts, &plan, true)) return W4A8_ERR_SHAPE;
    return launch_linear_tcgen05(Xq, tok_scale, blob, L, bias, M, static_cast<__nv_bfloat16 *>(Y),
                                 acc, static_cast<uint8_t *>(workspace), plan, st, zp);
}

}  // namespace

extern "C" {

size_t w4a8_packed_bytes(int N, int K, int group_size)
{
    if (!shape_ok(N, K, group_size)) return 0;
    return make_layout(N, K, group_size).total_bytes;
}

w4a8_status w4a8_pack_weights(const void *W_f16, const float *s_in, int N, int K, int group_size,
                              float clip, void *packed, size_t packed_bytes, void *stream)
{
    return w4a8_pack_weights_fmt(W_f16, s_in, N, K, group_size, clip, 1, packed, packed_bytes,
                                 stream);
}

w4a8_status w4a8_pack_weights_fmt(const void *W_f16, const float *s_in, int N, int K,
                                  int group_size, float clip, int level_shift, void *packed,
                                  size_t packed_bytes, void *stream)
{
    return w4a8_pack_weights_bits(W_f16, s_in, N, K, group_size, clip, 4, level_shift, packed,
                                  packed_bytes, stream);
}

size_t w4a8_packed_bytes_bits(int N, int K, int group_size, int bits)
{
    if (!shape_ok(N, K, group_size) || !bits_ok(bits)) return 0;
    return make_layout(N, K, group_size, 1, bits).total_bytes;
}

w4a8_status w4a8_pack_weights_bits(const void *W_f16, const float *s_in, int N, int K,
                                   int group_size, float clip, int bits, int level_shift,
                                   void *packed, size_t packed_bytes, void *stream)
{
    if (!W_f16 || !packed) return W4A8_ERR_NULL;
    if (!shape_ok(N, K, group_size) || !(clip > 0.0f && clip <= 1.0f) || !bits_ok(bits)) return W4A8_ERR_SHAPE;
    if (level_shift < 1 || level_shift > 3 || !depth_ok(K, level_shift, 127)) return W4A8_ERR_SHAPE;
    if (!aligned(W_f16, 16) || !aligned(s_in, 16) || !aligned(packed, 256)) return W4A8_ERR_ALIGN;
    const BlobLayout L = make_layout(N, K, group_size, level_shift, bits);
    if (packed_bytes < L.total_bytes) return W4A8_ERR_BUFFER_TOO_SMALL;
    const w4a8_status arch = check_arch();
    if (arch != W4A8_OK) return arch;
    const cudaError_t e = launch_pack(static_cast<const __half *>(W_f16), s_in, L, clip,
                                      static_cast<uint8_t *>(packed),
                                      static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_quantize_act(const void *X_f16, const float *inv_s_in, int M, int K,
                              int8_t *Xq, float *tok_scale, void *stream)
{
    if (!X_f16 || !Xq || !tok_scale) return W4A8_ERR_NULL;
    if (M < 1 || K < 128 || K % 128 != 0 || K >= (1 << 19)) return W4A8_ERR_SHAPE;
    if (!aligned(X_f16, 16) || !aligned(inv_s_in, 16) || !aligned(Xq, 16) ||
        !aligned(tok_scale, 4))
        return W4A8_ERR_ALIGN;
    const w4a8_status arch = check_arch();
    if (arch != W4A8_OK) return arch;
    const cudaError_t e =
        launch_quantize_act(static_cast<const __half *>(X_f16), inv_s_in, M, K, Xq, tok_scale,
                            static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_norm_quantize_act(const void *X_f16, const float *norm_weight,
                                   const float *norm_bias, int norm_kind, float eps, int M, int K,
                                   int8_t *Xq, float *tok_scale, void *stream)
{
    if (!X_f16 || !norm_weight || !Xq || !tok_scale) return W4A8_ERR_NULL;
    if (M < 1 || K < 128 || K % 128 != 0 || K > 16384) return W4A8_ERR_SHAPE;
    if (norm_kind != W4A8_NORM_RMS && norm_kind != W4A8_NORM_LAYER) return W4A8_ERR_SHAPE;
    if (!(eps > 0.0f)) return W4A8_ERR_SHAPE;
    if (!aligned(X_f16, 16) || !aligned(norm_weight, 16) || !aligned(norm_bias, 16) ||
        !aligned(Xq, 16) || !aligned(tok_scale, 4))
        return W4A8_ERR_ALIGN;
    const w4a8_status arch = check_arch();
    if (arch != W4A8_OK) return arch;
    const cudaError_t e = launch_norm_quantize_act(
        static_cast<const __half *>(X_f16), norm_weight, norm_bias, norm_kind == W4A8_NORM_LAYER, eps,
        M, K, Xq, tok_scale, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

size_t w4a8_linear_workspace_bytes_ex(int M, int N, int K, int group_size, const w4a8_opts *opts)
{
    if (!shape_ok(N, K, group_size) || M < 1 || !opts_ok(opts)) return 0;
    if (opts && opts->path == W4A8_PATH_SIMPLE) return sizeof(StatusBlock);
    LinearPlan plan;
    const BlobLayout L = make_layout(N, K, group_size, shift_of(opts), bits_of(opts));
    if (use_gemv(M, L, opts)) {
        if (M > gemv_max_tokens()) return 0;
        if (L.bits == 3 && gemv_row_slab_warps(M, L, opts ? opts->decode_warps : 0) == 0) return 0;
        gemv_plan(M, L, &plan);
        return plan.workspace_bytes;
    }
    if (!make_plan(M, L, opts, &plan, true)) return 0;
    return plan.workspace_bytes;
}

size_t w4a8_linear_workspace_bytes(int M, int N, int K, int group_size)
{
    return w4a8_linear_workspace_bytes_ex(M, N, K, group_size, nullptr);
}

w4a8_status w4a8_linear_plan(int M, int N, int K, int group_size, const w4a8_opts *opts, int *out)
{
    if (!out) return W4A8_ERR_NULL;
    if (!shape_ok(N, K, group_size) || M < 1 || !opts_ok(opts)) return W4A8_ERR_SHAPE;
    const BlobLayout L = make_layout(N, K, group_size, shift_of(opts), bits_of(opts));
    out[0] = out[1] = out[2] = out[3] = 0;
    out[4] = 1;
    if (opts && opts->path == W4A8_PATH_SIMPLE) {
        out[0] = W4A8_PATH_SIMPLE;
        return W4A8_OK;
    }
    LinearPlan plan;
    if (use_gemv(M, L, opts)) {
        if (M > gemv_max_tokens()) return W4A8_ERR_SHAPE;
        gemv_plan(M, L, &plan);
        const int warps = gemv_row_slab_warps(M, L, opts ? opts->decode_warps : 0);
        out[0] = W4A8_PATH_GEMV;
        out[2] = warps ? 1 : plan.split_k;
        out[3] = warps;
        return W4A8_OK;
    }
    if (!make_plan(M, L, opts, &plan, true)) return W4A8_ERR_SHAPE;
    out[0] = W4A8_PATH_TCGEN05;
    out[1] = plan.tok_tile;
    out[2] = plan.split_k;
    out[3] = plan.decode_warps;
    out[4] = plan.cluster;
    return W4A8_OK;
}

w4a8_status w4a8_workspace_init(void *workspace, size_t workspace_bytes, void *stream)
{
    if (!workspace) return W4A8_ERR_NULL;
    if (!aligned(workspace, 256)) return W4A8_ERR_ALIGN;
    if (workspace_bytes < sizeof(StatusBlock)) return W4A8_ERR_BUFFER_TOO_SMALL;
    const cudaError_t e =
        cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_linear(const int8_t *Xq, const float *tok_scale, const void *packed,
                        const float *bias, int M, int N, int K, int group_size, void *Y_bf16,
                        void *workspace, size_t workspace_bytes, void *stream)
{
    if (!Y_bf16) return W4A8_ERR_NULL;
    return linear_common(Xq, tok_scale, packed, bias, M, N, K, group_size, Y_bf16, nullptr,
                         workspace, workspace_bytes, stream, nullptr);
}

w4a8_status w4a8_linear_ex(const int8_t *Xq, const float *tok_scale, const void *packed,
                           const float *bias, int M, int N, int K, int group_size, void *Y_bf16,
                           void *workspace, size_t workspace_bytes, void *stream,
                           const w4a8_opts *opts)
{
    if (!Y_bf16) return W4A8_ERR_NULL;
    return linear_common(Xq, tok_scale, packed, bias, M, N, K, group_size, Y_bf16, nullptr,
                         workspace, workspace_bytes, stream, opts);
}

size_t w4a8_quantize_linear_workspace_bytes(int M, int N, int K, int group_size)
{
    if (!shape_ok(N, K, group_size) || M < 1 || M > gemv_max_tokens()) return 0;
    LinearPlan plan;
    gemv_plan(M, make_layout(N, K, group_size), &plan);
    // behind the kernel's own scratch: room for the INT8 tokens and their steps, used when the
    // quantizer runs as a launch of its own (see gemv_quantize_inside)
    return align_up(plan.workspace_bytes, 256) + align_up((size_t)M * K, 256) + 256;
}

w4a8_status w4a8_quantize_linear(const void *X_f16, const float *inv_s_in, const void *packed,
                                 const float *bias, int M, int N, int K, int group_size,
                                 void *Y_bf16, void *workspace, size_t workspace_bytes,
                                 void *stream)
{
    if (!X_f16 || !packed || !Y_bf16 || !workspace) return W4A8_ERR_NULL;
    if (!shape_ok(N, K, group_size) || M < 1 || M > gemv_max_tokens()) return W4A8_ERR_SHAPE;
    if (!depth_ok(K, 1, 127)) return W4A8_ERR_SHAPE;
    if (!aligned(X_f16, 16) || !aligned(inv_s_in, 16) || !aligned(bias, 4) ||
        !aligned(Y_bf16, 16) || !aligned(packed, 256) || !aligned(workspace, 256))
        return W4A8_ERR_ALIGN;
    const BlobLayout L = make_layout(N, K, group_size);
    LinearPlan plan;
    gemv_plan(M, L, &plan);
    if (workspace_bytes < w4a8_quantize_linear_workspace_bytes(M, N, K, group_size))
        return W4A8_ERR_BUFFER_TOO_SMALL;
    const w4a8_status arch = check_arch();
    if (arch != W4A8_OK) return arch;
    if (!gemv_quantize_inside(M, L)) {
        // several waves of CTAs: quantize once, in front, into the tail of the workspace
        uint8_t *ws = static_cast<uint8_t *>(workspace);
        int8_t *Xq = reinterpret_cast<int8_t *>(ws + align_up(plan.workspace_bytes, 256));
        float *tok = reinterpret_cast<float *>(ws + align_up(plan.workspace_bytes, 256) +
                                               align_up((size_t)M * K, 256));
        if (launch_quantize_act(static_cast<const __half *>(X_f16), inv_s_in, M, K, Xq, tok,
                                static_cast<cudaStream_t>(stream)) != cudaSuccess)
            return W4A8_ERR_CUDA;
        return launch_linear_gemv(Xq, tok, static_cast<const uint8_t *>(packed), L, bias, M,
                                  static_cast<__nv_bfloat16 *>(Y_bf16), nullptr, ws, plan,
                                  static_cast<cudaStream_t>(stream));
    }
    return launch_linear_gemv(nullptr, nullptr, static_cast<const uint8_t *>(packed), L, bias, M,
                              static_cast<__nv_bfloat16 *>(Y_bf16), nullptr,
                              static_cast<uint8_t *>(workspace), plan,
                              static_cast<cudaStream_t>(stream), ZeroPoint(),
                              static_cast<const __half *>(X_f16), inv_s_in);
}

// ---- gate / up projections with the gated unit in the epilogue ----
static bool swiglu_plan(int M, int F, int K, int group, BlobLayout *L, LinearPlan *plan)
{
    if (F < 8 || F % 8 != 0 || M < 1 || !shape_ok(2 * F, K, group)) return false;   // (bulk stores: rows of 16-byte multiples)
    *L = make_layout(2 * F, K, group);
    w4a8_opts o = {};
    o.path = W4A8_PATH_TCGEN05;
    o.split_k = 1;                      // the epilogue pairs rows inside one accumulator tile
    if (!make_plan(M, *L, &o, plan)) return false;
    plan->swiglu = 1;
    return true;
}

size_t w4a8_linear_swiglu_workspace_bytes(int M, int F, int K, int group_size)
{
    BlobLayout L;
    LinearPlan plan;
    return swiglu_plan(M, F, K, group_size, &L, &plan) ? plan.workspace_bytes : 0;
}

w4a8_status w4a8_linear_swiglu(const int8_t *Xq, const float *tok_scale, const void *packed_gate_up,
                               const float *bias_gate_up, int M, int F, int K, int group_size,
                               void *H_f16, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!Xq || !tok_scale || !packed_gate_up || !H_f16 || !workspace) return W4A8_ERR_NULL;
    BlobLayout L;
    LinearPlan plan;
    if (!swiglu_plan(M, F, K, group_size, &L, &plan) || !depth_ok(K, 1, 127)) return W4A8_ERR_SHAPE;
    if (!aligned(Xq, 16) || !aligned(tok_scale, 4) || !aligned(bias_gate_up, 4) || !aligned(H_f16, 16) ||
        !aligned(packed_gate_up, 256) || !aligned(workspace, 256))
        return W4A8_ERR_ALIGN;
    if (workspace_bytes < plan.workspace_bytes) return W4A8_ERR_BUFFER_TOO_SMALL;
    const w4a8_status arch = check_arch();
    if (arch != W4A8_OK) return arch;
    return launch_linear_tcgen05(Xq, tok_scale, static_cast<const uint8_t *>(packed_gate_up), L,
                                 bias_gate_up, M, static_cast<__nv_bfloat16 *>(H_f16), nullptr,
                                 static_cast<uint8_t *>(workspace), plan,
                                 static_cast<cudaStream_t>(stream));
}

// ---- attention value path (W4A8V4): P * V with channel-wise dINT4 values ----
w4a8_status w4a8_pack_value(const void *V_f16, int S, int H, int D, float clip, void *packed,
                            size_t packed_bytes, void *stream)
{
    if (!V_f16 || !packed) return W4A8_ERR_NULL;
    if (D != kTileN || H < 1 || H > 4096 || !shape_ok(H * D, S, 0) || !(clip > 0.0f && clip <= 1.0f))
        return W4A8_ERR_SHAPE;
    if (!depth_ok(S, 1, 127)) return W4A8_ERR_SHAPE;
    if (!aligned(V_f16, 16) || !aligned(packed, 256)) return W4A8_ERR_ALIGN;
    const BlobLayout L = make_layout(H * D, S, 0);
    if (packed_bytes < L.total_bytes) return W4A8_ERR_BUFFER_TOO_SMALL;
    const w4a8_status arch = check_arch();
    if (arch != W4A8_OK) return arch;
    const cudaError_t e = launch_pack_transposed(static_cast<const __half *>(V_f16), L, clip,
                                                 static_cast<uint8_t *>(packed),
                                                 static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

size_t w4a8_attn_pv_workspace_bytes(int T, int S, int H, int D)
{
    if (D != kTileN || H < 1 || T < 1 || !shape_ok(H * D, S, 0)) return 0;
    LinearPlan plan;
    w4a8_opts o = {};
    o.path = W4A8_PATH_TCGEN05;
    if (!make_plan(T, make_layout(H * D, S, 0), &o, &plan)) return 0;
    return plan.workspace_bytes;
}

w4a8_status w4a8_attn_pv(const int8_t *Pq, const float *p_scale, const void *packed, int T, int S,
                         int H, int D, void *O_bf16, void *workspace, size_t workspace_bytes,
                         void *stream)
{
    if (!Pq || !p_scale || !packed || !O_bf16 || !workspace) return W4A8_ERR_NULL;
    if (D != kTileN || H < 1 || T < 1 || !shape_ok(H * D, S, 0) || !depth_ok(S, 1, 127))
        return W4A8_ERR_SHAPE;
    if (!aligned(Pq, 16) || !aligned(p_scale, 4) || !aligned(O_bf16, 16) || !aligned(packed, 256) ||
        !aligned(workspace, 256))
        return W4A8_ERR_ALIGN;
    const BlobLayout L = make_layout(H * D, S, 0);
    LinearPlan plan;
    w4a8_opts o = {};
    o.path = W4A8_PATH_TCGEN05;
    if (!make_plan(T, L, &o, &plan)) return W4A8_ERR_SHAPE;
    if (workspace_bytes < plan.workspace_bytes) return W4A8_ERR_BUFFER_TOO_SMALL;
    const w4a8_status arch = check_arch();
    if (arch != W4A8_OK) return arch;
    plan.batched = 1;            // head h = row tile h reads its own [T][S] block of Pq and p_scale
    return launch_linear_tcgen05(Pq, p_scale, static_cast<const uint8_t *>(packed), L, nullptr, T,
                                 static_cast<__nv_bfloat16 *>(O_bf16), nullptr,
                                 static_cast<uint8_t *>(workspace), plan,
                                 static_cast<cudaStream_t>(stream));
}

w4a8_status w4a8_linear_acc_i32(const int8_t *Xq, const void *packed, int M, int N, int K,
                                int group_size, int32_t *acc, void *workspace,
                                size_t workspace_bytes, void *stream, const w4a8_opts *opts)
{
    if (!acc) return W4A8_ERR_NULL;
    return linear_common(Xq, nullptr, packed, nullptr, M, N, K, group_size, nullptr, acc,
                         workspace, workspace_bytes, stream, opts);
}

w4a8_status w4a8_quantize_act_asym(const void *X_f16, const float *inv_s_in, int M, int K,
                                   int8_t *Xq, float *tok_scale, int32_t *tok_zero, void *stream)
{
    if (!X_f16 || !Xq || !tok_scale || !tok_zero) return W4A8_ERR_NULL;
    if (M < 1 || K < 128 || K % 128 != 0 || K >= (1 << 19)) return W4A8_ERR_SHAPE;
    if (!aligned(X_f16, 16) || !aligned(inv_s_in, 16) || !aligned(Xq, 16) ||
        !aligned(tok_scale, 4) || !aligned(tok_zero, 4))
        return W4A8_ERR_ALIGN;
    const w4a8_status arch = check_arch();
    if (arch != W4A8_OK) return arch;
    const cudaError_t e =
        launch_quantize_act_asym(static_cast<const __half *>(X_f16), inv_s_in, M, K, Xq, tok_scale,
                                 tok_zero, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_weight_rowsum(const void *packed, int N, int K, int group_size, int32_t *rowsum,
                               void *stream)
{
    if (!packed || !rowsum) return W4A8_ERR_NULL;
    if (!shape_ok(N, K, group_size)) return W4A8_ERR_SHAPE;
    if (!aligned(packed, 256) || !aligned(rowsum, 4)) return W4A8_ERR_ALIGN;
    const w4a8_status arch = check_arch();
    if (arch != W4A8_OK) return arch;
    const cudaError_t e =
        launch_weight_rowsum(static_cast<const uint8_t *>(packed), make_layout(N, K, group_size),
                             rowsum, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_linear_asym(const int8_t *Xq, const float *tok_scale, const int32_t *tok_zero,
                             const void *packed, const int32_t *rowsum, const float *bias, int M,
                             int N, int K, void *Y_bf16, int32_t *acc, void *workspace,
                             size_t workspace_bytes, void *stream, const w4a8_opts *opts)
{
    if (!tok_zero || !rowsum) return W4A8_ERR_NULL;
    if (!aligned(tok_zero, 4) || !aligned(rowsum, 4)) return W4A8_ERR_ALIGN;
    ZeroPoint zp;
    zp.tok_zero = tok_zero;
    zp.rowsum = rowsum;
    return linear_common(Xq, tok_scale, packed, bias, M, N, K, 0, Y_bf16, acc, workspace,
                         workspace_bytes, stream, opts, zp);
}

w4a8_status w4a8_linear_asym_group(const int8_t *Xq, const float *tok_scale, const int32_t *tok_zero,
                                   const void *packed, const int32_t *rowsum, const float *bias,
                                   int M, int N, int K, int group_size, void *Y_bf16, int32_t *acc,
                                   void *workspace, size_t workspace_bytes, void *stream,
                                   const w4a8_opts *opts)
{
    if (!tok_zero || !rowsum) return W4A8_ERR_NULL;
    if (!aligned(tok_zero, 4) || !aligned(rowsum, 4)) return W4A8_ERR_ALIGN;
    ZeroPoint zp;
    zp.tok_zero = tok_zero;
    zp.rowsum = rowsum;
    return linear_common(Xq, tok_scale, packed, bias, M, N, K, group_size, Y_bf16, acc, workspace,
                         workspace_bytes, stream, opts, zp);
}

w4a8_status w4a8_unpack_codes(const void *packed, int N, int K, int group_size, uint8_t *codes,
                              float *scales, uint8_t *zeros, void *stream)
{
    return w4a8_unpack_codes_bits(packed, N, K, group_size, 4, codes, scales, zeros, stream);
}

w4a8_status w4a8_unpack_codes_bits(const void *packed, int N, int K, int group_size, int bits,
                                   uint8_t *codes, float *scales, uint8_t *zeros, void *stream)
{
    if (!packed || !codes || !scales || !zeros) return W4A8_ERR_NULL;
    if (!shape_ok(N, K, group_size) || !bits_ok(bits)) return W4A8_ERR_SHAPE;
    if (!aligned(packed, 256) || !aligned(scales, 4)) return W4A8_ERR_ALIGN;
    const w4a8_status arch = check_arch();
    if (arch != W4A8_OK) return arch;
    const cudaError_t e =
        launch_unpack(static_cast<const uint8_t *>(packed), make_layout(N, K, group_size, 1, bits), codes,
                      scales, zeros, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_poll_status(void *workspace, void *stream)
{
    if (!workspace) return W4A8_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return W4A8_ERR_CUDA;
    int host[3] = {0, 0, 0};
    if (cudaMemcpy(host, workspace, sizeof(host), cudaMemcpyDeviceToHost) != cudaSuccess)
        return W4A8_ERR_CUDA;
    if (host[0] == 0) return W4A8_OK;
    if (cudaMemset(workspace, 0, sizeof(StatusBlock)) != cudaSuccess) return W4A8_ERR_CUDA;
    return host[0] == W4A8_ERR_BAD_BLOB ? W4A8_ERR_BAD_BLOB : W4A8_ERR_TIMEOUT;
}

void w4a8_dint4_table(int z, int8_t *out) { w4a8_dint4_table_fmt(z, 1, out); }

void w4a8_dint4_table_fmt(int z, int level_shift, int8_t *out)
{
    for (int c = 0; c < 16; ++c) out[c] = (int8_t)dint4_level(c, z, level_shift);
}

void w4a8_dint_table_bits(int z, int bits, int level_shift, int8_t *out)
{
    for (int c = 0; c < 16; ++c) out[c] = c < (1 << bits) ? (int8_t)dint_level(c, z, level_shift, bits) : 0;
}

const char *w4a8_version(void) { return "w4a8-dint 0.1 (sm_100a)"; }

}  // extern "C"
