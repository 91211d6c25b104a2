/*
 * w4a8.h - C ABI of the B200 (sm_100a) W4A8-dINT quantized linear layer.
 *
 * The layer computes  Y = Q(diag(s)^-1 X) * Q(W diag(s))^T  (+ bias)  of
 * arXiv 2311.05161, Eq. 1, with
 *   - weights W[N][K] (N output features, K input features) quantized per output
 *     channel, or per group of 128 input features, to the 4-bit dINT format of
 *     Section 4.2 (Eq. 5 quantize, Eq. 6 dequantize): integer levels 0..13 plus two
 *     special codes worth +s/2 and -s/2;
 *   - activations X[M][K] (M tokens) quantized per token to INT8 (Appendix A.1,
 *     "token-wise quantization for activations"), symmetric absmax variant;
 *   - an exact INT8 x INT8 -> INT32 contraction on the tensor cores, in which a dINT
 *     code stands for the integer 2 * (value / s), so the half-step levels stay whole;
 *   - an FP32 rescale by (token step) x (weight step / 2), optional FP32 bias, BF16 out.
 *
 * General rules
 *   - Every pointer is a DEVICE pointer owned by the caller unless marked "host".
 *   - Row-major everywhere.  K % 128 == 0, N % 8 == 0, M >= 1, K < 2^19.
 *   - group_size is 0 (one step size and zero-point per output channel) or 128.
 *   - Base pointers must be 16-byte aligned, `packed` and `workspace` 256-byte aligned.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  All work
 *     is enqueued on it; no call synchronizes the device except w4a8_poll_status.
 *   - The library allocates no device memory and keeps no device state between calls (the one
 *     exception is the fixed scratch array of w4a8_linear_static, see there).
 *   - Every call validates its arguments first and launches nothing when validation
 *     fails.  Inputs holding NaN or Inf are a precondition violation.
 *   - There is no CPU or other-architecture fallback: a device that is not compute
 *     capability 10.x makes the compute calls return W4A8_ERR_UNSUPPORTED_ARCH.
 */
#ifndef W4A8_H_
#define W4A8_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    W4A8_OK = 0,
    W4A8_ERR_NULL = 1,              /* a required pointer is NULL */
    W4A8_ERR_SHAPE = 2,             /* M, N, K, group_size or an option outside the rules */
    W4A8_ERR_ALIGN = 3,             /* a pointer breaks the alignment rule */
    W4A8_ERR_BUFFER_TOO_SMALL = 4,  /* packed_bytes / workspace_bytes below the query */
    W4A8_ERR_UNSUPPORTED_ARCH = 5,  /* current device is not sm_100 */
    W4A8_ERR_CUDA = 6,              /* a CUDA runtime or driver call failed */
    W4A8_ERR_TIMEOUT = 7,           /* a bounded wait inside a kernel ran out */
    W4A8_ERR_BAD_BLOB = 8           /* `packed` does not hold a blob of this N, K, group */
} w4a8_status;

/* Which kernel w4a8_linear_ex runs.  AUTO picks by shape. */
typedef enum {
    W4A8_PATH_AUTO = 0,
    W4A8_PATH_SIMPLE = 1,   /* one thread per output, CUDA cores: slow cross-check */
    W4A8_PATH_TCGEN05 = 2,  /* TMA + in-register dINT decode + tcgen05 kind::i8 MMA */
    W4A8_PATH_GEMV = 3      /* weight-streaming CUDA-core kernel, M <= 4 tokens (AUTO picks it for M <= 2) */
} w4a8_path;

typedef struct {
    int path;        /* w4a8_path */
    int split_k;     /* 0 = automatic; else number of K slices (tcgen05 path) */
    int tok_tile;    /* 0 = automatic; else tokens per tile: 16, 32, 64, 128, 192 or 256 */
    int decode_warps;/* 0 = automatic; else warps that expand codes to INT8: 4, 8, 12 or 16 (with
                        W4A8_PATH_GEMV: the warps of a CTA that owns a slab of rows: 4, 8, 16
                        or 32) */
    int level_shift; /* special value of the blob = step / 2^level_shift: 0 or 1 (the paper's
                        step/2), 2 or 3 (w4a8_pack_weights_fmt); must match the blob */
    int cluster;     /* 0 = automatic: form 3 or 5 (form 4 from K = 32768 on) with offset tables for
                        1024 tokens and more on layers of at least 8192 x 8192 when the shape
                        allows it (and decode_warps and offset_tables are 0), else form 1;
                        else the form of the tensor-core kernel:
                        1 = one CTA per cluster, one row tile per CTA;
                        2 = sharing pair (token tiles of 128 and more, symmetric activations
                            when the weights are grouped): two CTAs work on two token tiles of
                            the same weight rows and each expands half of every code tile for both;
                        3 = MMA pair (token tile 256, per-channel 4-bit weights, even numbers
                            of 128-row tiles and of k-blocks per K slice, 8 or 16 decode warps): two
                            CTAs on two row tiles and one token tile issue every MMA as one
                            256-row instruction, each loads half of the tokens;
                        4 = two row tiles per CTA (token tile 256, per-channel 4-bit weights, an
                            even number of 128-row tiles, 16 decode warps): one CTA
                            multiplies two row tiles by the same token buffer;
                        5 = form 3 with three k-blocks per barrier round instead of two (numbers
                            of k-blocks per K slice that are multiples of three, 16 decode warps).
                        Same bits in every form; a form that does not fit the call is refused
                        with W4A8_ERR_SHAPE. */
    int debug_wait_ms;   /* test hook, 0 = off: limit of every bounded wait inside the tensor-core
                            kernel in milliseconds (normally 2 s) */
    int debug_skip_load; /* test hook, 0 = off: the copy thread of every CTA leaves out the token
                            load of its k-block number debug_skip_load - 1, so that a wait runs
                            out and the kernel reports W4A8_ERR_TIMEOUT.  Both hooks are refused
                            (W4A8_ERR_SHAPE) unless the library was built with W4A8_DEBUG_HOOKS,
                            and only w4a8_linear_ex with W4A8_PATH_TCGEN05 takes them */
    int bits;        /* code width of the blob: 0 or 4 (dINT4), or 3 (dINT3, packed by
                        w4a8_pack_weights_bits); must match the blob.  3-bit blobs run on the
                        tensor-core kernel (any M), the row-slab form of the weight-streaming
                        kernel (one or two tokens, layers of 3072 rows and more) or the simple
                        kernel, with symmetric activations */
    int offset_tables; /* 0 = off (on with the automatic MMA pair, see cluster); 1 = the
                        tensor-core kernel expands codes through level tables
                        stored with an offset (fewer logic instructions per code) and takes the
                        offset out again with the tokens' sums, which a small kernel in front
                        computes into the workspace.  Per-channel 4-bit weights, level_shift
                        1 or 2.  Same bits as without. */
    int tok_run;     /* 0 = automatic; else the token tiles per run in the order in which the
                        tensor-core kernel's CTAs take their work: inside a run the token tile
                        changes fastest, then the 128-row tile (1: every token tile walks through
                        all row tiles; many: CTAs that work side by side read the same codes).
                        The automatic choice streams whichever operand does not fit in L2 once.
                        Runs longer than one exist for per-channel 4-bit weights with token tiles
                        of 128 and more; elsewhere the field is accepted and has no effect.
                        Same bits either way. */
} w4a8_opts;

/* Bytes of the packed-weight blob for an [N][K] matrix; 0 if the shape is invalid.
 * Blob = 256-byte header, step sizes FP32 [G][Npad], zero-points u8 [G][Npad], then the
 * codes in 8 KiB tiles of 128 output rows x 128 input features (G = 1 or K/128,
 * Npad = N rounded up to 128).  Inside a tile, byte q*2048 + r*16 + j holds the codes of
 * row r for k = 32 q + 2 j (low nibble) and 32 q + 2 j + 1 (high nibble).  The blob can be
 * copied, saved and reloaded byte for byte. */
size_t w4a8_packed_bytes(int N, int K, int group_size);

/* Weight side of Eq. 1 with the dINT4 quantizer of Eq. 5 (offline, once per layer).
 *   W_f16   [N][K] IEEE binary16.
 *   s_in    [K] FP32 per-input-channel scale s of Eq. 1, or NULL (all ones).
 *   clip    ratio in (0, 1] applied to both ends of the Min-Max range (Appendix A.4
 *           mentions an extra weight clipping after the scale search); 1.0f = Min-Max.
 *   packed  out, packed_bytes >= w4a8_packed_bytes(N, K, group_size).
 * Per row (or per 128-wide group): w' = W * s, lo = min(0, min w') * clip,
 * hi = max(0, max w') * clip, step = (hi - lo) / 13 (1 if zero),
 * zero-point = clamp(rint(-lo / step), 0, 13), codes by Eq. 5 with c1 = 14, c2 = 15. */
w4a8_status w4a8_pack_weights(const void *W_f16, const float *s_in, int N, int K,
                              int group_size, float clip, void *packed,
                              size_t packed_bytes, void *stream);

/* w4a8_pack_weights with another special value: c = step / 2^level_shift, level_shift 1 (the
 * paper's step/2, Eq. 5 / Eq. 6), 2 or 3 (step/4, step/8: the sweep of Appendix A.5).  A
 * value becomes +-c when c/2 < |x| <= (c + step)/2 (the midpoints towards 0 and towards
 * +-step; Eq. 5's s/4 and 3s/4 for level_shift 1).  The levels are then integers in units of
 * c: 2^level_shift (code - z), +1, -1, and the linear calls rescale by step / 2^level_shift.
 * Linear calls on such a blob pass the same level_shift in their options: w4a8_linear_ex,
 * w4a8_linear_acc_i32, w4a8_linear_asym; a mismatch is reported as W4A8_ERR_BAD_BLOB.
 * K is limited so that K * 127 * 13 * 2^level_shift < 2^31. */
w4a8_status w4a8_pack_weights_fmt(const void *W_f16, const float *s_in, int N, int K,
                                  int group_size, float clip, int level_shift, void *packed,
                                  size_t packed_bytes, void *stream);

/* The same quantizer for the b-bit dINT format of Section 4.2 with b = 3 or 4: p = 2^b - 3
 * uniform steps, integer codes 0..p, code p + 1 = +c, code p + 2 = -c (b = 3, the format of
 * Tables 10-11: codes 0..5, 6 = +c, 7 = -c; step = range / 5, zero-point 0..5).  A 3-bit blob
 * has the layout of the 4-bit one except for its code tiles: 6144 bytes per 128 x 128 tile
 * (0.375 byte per weight); per 32-k quarter and row three 32-bit words hold 32 codes - nibble j
 * of word w carries the code of k = 8 w + j in its low three bits, and the spare top bits of
 * the nibbles j of words 0, 1, 2 are bits 0, 1, 2 of the code of k = 24 + j; word w of row r of
 * quarter q is at byte q * 1536 + w * 512 + r * 4 of the tile.
 * Linear calls on a 3-bit blob name bits = 3 (and the level_shift) in their options. */
size_t w4a8_packed_bytes_bits(int N, int K, int group_size, int bits);
w4a8_status w4a8_pack_weights_bits(const void *W_f16, const float *s_in, int N, int K,
                                   int group_size, float clip, int bits, int level_shift,
                                   void *packed, size_t packed_bytes, void *stream);

/* Activation side of Eq. 1, token-wise INT8 (Appendix A.1), every forward pass.
 *   X_f16     [M][K] IEEE binary16.
 *   inv_s_in  [K] FP32 reciprocal of the Eq. 1 scale, or NULL.
 *   Xq        out [M][K] INT8;  tok_scale out [M] FP32.
 * Per token: x' = X * inv_s, amax = max |x'|, tok_scale = amax / 127,
 * q = clamp(rint(x' * (127 / amax)), -127, 127); an all-zero token gives scale 0. */
w4a8_status w4a8_quantize_act(const void *X_f16, const float *inv_s_in, int M, int K,
                              int8_t *Xq, float *tok_scale, void *stream);

/* The activation side of Eq. 1 where it lives in a decoder layer: inside the normalisation in
 * front of the matmul (Fig. 1(a), Section 3.1 - the reciprocal scale diag(s)^-1 is merged into
 * the normalisation's weight and bias), followed at once by the token-wise INT8 quantizer
 * (Appendix A.1).  One pass over X: the normalised FP16 tensor is never written.
 *   X_f16        [M][K] IEEE binary16, the layer input before the normalisation.
 *   norm_weight  [K] FP32, the normalisation's weight times the reciprocal Eq. 1 scale.
 *   norm_bias    [K] FP32 likewise, or NULL.
 *   norm_kind    W4A8_NORM_RMS:   x' = (x / sqrt(mean(x^2) + eps)) * weight (+ bias)
 *                W4A8_NORM_LAYER: x' = ((x - mean(x)) / sqrt(var(x) + eps)) * weight (+ bias)
 *   eps          > 0.   K <= 16384 (the hidden sizes a normalisation sees).
 *   Xq, tok_scale  out, as from w4a8_quantize_act applied to x'.
 * Precision: the token statistics (sums, mean, variance, reciprocal root) in binary64, rounded
 * once to binary32; everything per element in binary32, one rounding per operation. */
typedef enum { W4A8_NORM_RMS = 0, W4A8_NORM_LAYER = 1 } w4a8_norm;
w4a8_status w4a8_norm_quantize_act(const void *X_f16, const float *norm_weight,
                                   const float *norm_bias, int norm_kind, float eps, int M, int K,
                                   int8_t *Xq, float *tok_scale, void *stream);

/* Scratch bytes w4a8_linear needs for this shape (always >= 256: the first 256 bytes
 * hold the status block read by w4a8_poll_status).  The caller zero-fills the workspace
 * once after allocating it (w4a8_workspace_init); calls that end without a reported failure
 * leave it ready for reuse (after a failure: see w4a8_poll_status).  Calls
 * that may overlap on the device need separate workspaces.  The _ex form answers for
 * explicit options (NULL = automatic); 0 means the shape or the options are invalid. */
size_t w4a8_linear_workspace_bytes(int M, int N, int K, int group_size);
size_t w4a8_linear_workspace_bytes_ex(int M, int N, int K, int group_size,
                                      const w4a8_opts *opts);

/* Host: which kernel and tiling w4a8_linear_ex would run for this shape and these options
 * (NULL = automatic, i.e. what w4a8_linear runs), without touching a device.  `out` is a host
 * array of 5: out[0] = w4a8_path; out[1] = tokens per tile (tensor-core kernel, else 0);
 * out[2] = K slices; out[3] = warps that expand codes (tensor-core kernel) or warps of a
 * row-slab CTA (weight-streaming kernel; 0 = its K-sliced variant); out[4] = cluster form (see w4a8_opts.cluster).
 * The plan follows the SM
 * count of the current device (148 when there is none).  Eq. 1 fixes the result, not the plan:
 * this call only reports the choice, e.g. where the weight-streaming kernel hands over to the
 * tensor-core kernel as M grows. */
w4a8_status w4a8_linear_plan(int M, int N, int K, int group_size, const w4a8_opts *opts, int *out);

/* Zero-fill a workspace (enqueued on `stream`). */
w4a8_status w4a8_workspace_init(void *workspace, size_t workspace_bytes, void *stream);

/* The quantized matmul of Eq. 1 with the dINT dequantization of Eq. 6 folded in.
 *   Xq, tok_scale  as written by w4a8_quantize_act ([M][K] INT8, [M] FP32).
 *   packed         as written by w4a8_pack_weights for the same N, K, group_size.
 *   bias           [N] FP32 or NULL.
 *   Y_bf16         out [M][N] bfloat16.
 * acc[m][n](g) = sum_k Xq[m][k] * t2(code[n][k]),  t2 = 2 (code - z) | +1 | -1   (INT32)
 * per channel : y = (float(acc) * tok_scale[m]) * (0.5 * step[n])
 * group 128   : y = (sum_g float(acc_g) * (0.5 * step[g][n])) * tok_scale[m]     (FP32)
 * then y += bias[n], rounded to BF16 nearest-even.
 * Returns W4A8_OK once the work is enqueued; kernel-side failures (a wait that ran out,
 * a blob that does not match) are reported by w4a8_poll_status. */
w4a8_status w4a8_linear(const int8_t *Xq, const float *tok_scale, const void *packed,
                        const float *bias, int M, int N, int K, int group_size,
                        void *Y_bf16, void *workspace, size_t workspace_bytes,
                        void *stream);

/* Same as w4a8_linear with the kernel, K split and token tile chosen by the caller
 * (opts == NULL behaves like w4a8_linear).  Unsupported combinations return
 * W4A8_ERR_SHAPE. */
w4a8_status w4a8_linear_ex(const int8_t *Xq, const float *tok_scale, const void *packed,
                           const float *bias, int M, int N, int K, int group_size,
                           void *Y_bf16, void *workspace, size_t workspace_bytes,
                           void *stream, const w4a8_opts *opts);

/* Decode form of the whole of Eq. 1 for one to four tokens: the token-wise activation
 * quantizer (Appendix A.1, as in w4a8_quantize_act) and the quantized matmul with the Eq. 6
 * dequantization (as in w4a8_linear) in ONE launch.  With so few tokens the layer is a single
 * scan of the packed weights, and a separate quantizer launch costs as much as a good part of
 * that scan; here every CTA of the weight-streaming kernel quantizes the tokens itself
 * (M * K elements, read from L2) while its first codes are on their way.
 *   X_f16     [M][K] IEEE binary16, 1 <= M <= 4 (else W4A8_ERR_SHAPE).
 *   inv_s_in  [K] FP32 reciprocal of the Eq. 1 scale, or NULL.
 *   packed    as written by w4a8_pack_weights (special value step/2) for N, K, group_size.
 *   bias      [N] FP32 or NULL.   Y_bf16  out [M][N] bfloat16.
 *   workspace >= w4a8_quantize_linear_workspace_bytes(M, N, K, group_size) bytes, zero-filled
 *             once (w4a8_workspace_init); same rules as for w4a8_linear.
 * It pays on layers of a few tens of megabytes of codes (the OPT-6.7B-shaped block: 45 -> 42 us
 * per step).  On a matrix so large that its CTAs come in several waves (170 MB of codes), each
 * wave would repeat the quantizer; there the call runs the quantizer as a launch of its own in
 * front, into the tail of the workspace (same results, two launches).
 * The result has the very bits of w4a8_quantize_act followed by w4a8_linear on the same
 * inputs; the INT8 tokens and their steps are not returned.  Kernel-side failures
 * are reported by w4a8_poll_status. */
size_t w4a8_quantize_linear_workspace_bytes(int M, int N, int K, int group_size);
w4a8_status w4a8_quantize_linear(const void *X_f16, const float *inv_s_in, const void *packed,
                                 const float *bias, int M, int N, int K, int group_size,
                                 void *Y_bf16, void *workspace, size_t workspace_bytes,
                                 void *stream);

/* w4a8_linear for callers that must not allocate device memory and therefore have no
 * workspace to pass: code running after a host framework has claimed the whole device for
 * its own pool (a cudaMalloc there fails or stalls the device), plug-ins whose host forbids
 * allocation once serving has started, and real-time loops that may not risk the implicit
 * synchronisation of an allocation.  The paper has no counterpart of this call; it is
 * w4a8_linear on the tensor-core kernel with its automatic plan (also for one or two
 * tokens, where w4a8_linear would pick the weight-streaming kernel), and it calls no
 * allocating routine.  Per-channel results have the bits of w4a8_linear; group-128 results
 * too wherever w4a8_linear runs the same kernel (three tokens and more), else they agree
 * within the FP32 reordering allowance of the group sums.
 *   The scratch is an 8 MiB array inside the library image (each GPU that loads the
 *   library holds it until the process ends).  Shapes whose plan needs more than that
 *   (large split-K cases; w4a8_linear_workspace_bytes tells) return
 *   W4A8_ERR_BUFFER_TOO_SMALL and launch nothing.
 *   The first call on each device looks up the array's device address; make that first
 *   call outside any stream capture.
 *   All calls on one device share the array: the call clears the part that must start at
 *   zero, on `stream`, before its kernel.  Two calls that can overlap on the GPU (different
 *   streams without an ordering between them) race on it and give undefined results.
 *   Failures inside the kernel are not reported through this call: poll them with
 *   w4a8_static_poll_status before the next call. */
w4a8_status w4a8_linear_static(const int8_t *Xq, const float *tok_scale, const void *packed,
                               const float *bias, int M, int N, int K, int group_size,
                               void *Y_bf16, void *stream);

/* Synchronizes `stream` and returns what the kernel of the last w4a8_linear_static call on the
 * current device reported (W4A8_OK, W4A8_ERR_TIMEOUT, W4A8_ERR_BAD_BLOB).  The next
 * w4a8_linear_static call clears that status, so poll before it.  Allocates nothing. */
w4a8_status w4a8_static_poll_status(void *stream);

/* ---- asymmetric token-wise activations (the paper's own activation quantizer) ----
 * Appendix A.1 quantizes activations token-wise with an asymmetric Min-Max quantizer; the
 * three calls below are that variant of the path, for per-output-channel weights
 * (group_size 0, the paper's W4A8 setting).
 *
 * Per token: x' = X * inv_s, lo = min(0, min x'), hi = max(0, max x'), d = hi - lo,
 * tok_scale = d / 255, r = 255 / d, zx = clamp(rint(-lo * r), 0, 255),
 * Q = clamp(rint(x' * r) + zx, 0, 255), so x' ~ tok_scale * (Q - zx); d = 0 gives scale 0.
 * The unsigned code and its zero-point are stored shifted by 128 so that the INT8 tensor
 * and CUDA-core paths take them unchanged:
 *   Xq        out [M][K] INT8  = Q - 128
 *   tok_scale out [M] FP32
 *   tok_zero  out [M] INT32    = zx - 128                                               */
w4a8_status w4a8_quantize_act_asym(const void *X_f16, const float *inv_s_in, int M, int K,
                                   int8_t *Xq, float *tok_scale, int32_t *tok_zero,
                                   void *stream);

/* Row sums of the doubled weight levels, rowsum[g][n] = sum over k in group g of
 * t2(code[n][k]) (INT32, [G][N]; G = 1 for per-channel weights): what a token's zero-point
 * multiplies.  Offline, once per packed layer. */
w4a8_status w4a8_weight_rowsum(const void *packed, int N, int K, int group_size,
                               int32_t *rowsum, void *stream);

/* The quantized matmul with asymmetric activations:
 *   acc[m][n] = sum_k (Q[m][k] - zx[m]) * t2(code[n][k])
 *             = sum_k Xq[m][k] * t2(code[n][k]) - tok_zero[m] * rowsum[n]          (INT32)
 *   y = (float(acc) * tok_scale[m]) * (0.5 * step[n]) + bias[n]  ->  bfloat16.
 * Xq, tok_scale, tok_zero as written by w4a8_quantize_act_asym; rowsum [N] as written by
 * w4a8_weight_rowsum; packed with group_size 0.  Y_bf16 and acc ([M][N] INT32, the sums
 * above) are outputs, either may be NULL but not both.  opts as in w4a8_linear_ex
 * (NULL = automatic); workspace as for w4a8_linear_ex with the same opts. */
w4a8_status w4a8_linear_asym(const int8_t *Xq, const float *tok_scale, const int32_t *tok_zero,
                             const void *packed, const int32_t *rowsum, const float *bias,
                             int M, int N, int K, void *Y_bf16, int32_t *acc, void *workspace,
                             size_t workspace_bytes, void *stream, const w4a8_opts *opts);

/* ---- gate and up projections of a gated feed-forward block with the unit in the epilogue ----
 * In a LLaMA-style block the two projections that read the same quantized input (gate and up)
 * feed h = silu(gate) * up, which is the next quantized matmul's input ("all matrix
 * multiplications in the Decoder layer", Appendix A.1): here both run as ONE quantized linear
 * layer over a weight matrix of 2 F rows in which row 2 i is row i of the gate projection and row
 * 2 i + 1 row i of the up projection (interleave, then w4a8_pack_weights), and the epilogue
 * writes h instead of the two BF16 outputs: per element the FP32 value of w4a8_linear before its
 * BF16 rounding (g for the even row, u for the odd row, bias included), then
 *   h = (g / (1 + exp(-g))) * u   in FP32, rounded to binary16.
 * H_f16 [M][F] is what w4a8_quantize_act takes next.  F % 8 == 0.  bias_gate_up [2 F]
 * interleaved like the rows, or NULL.  workspace >= w4a8_linear_swiglu_workspace_bytes(...),
 * zero-filled once.  The exponential is the GPU's fast one: results agree with a binary64
 * evaluation of the formula to one binary16 step. */
size_t w4a8_linear_swiglu_workspace_bytes(int M, int F, int K, int group_size);
w4a8_status w4a8_linear_swiglu(const int8_t *Xq, const float *tok_scale, const void *packed_gate_up,
                               const float *bias_gate_up, int M, int F, int K, int group_size,
                               void *H_f16, void *workspace, size_t workspace_bytes, void *stream);

/* ---- attention value path: "W4A8V4" (Section 5; Appendix A.1: channel-wise 4-bit Value) ----
 * The product of the attention map and the values, O[t][h][d] = sum_s P[h][t][s] V[s][h][d], with
 * V quantized to dINT4 per channel (h, d) - the dimension along which the partial sums
 * accumulate is the sequence s, so one step size and zero-point per channel factor out of the sum
 * - and the attention map quantized token-wise to INT8 like every other activation.  With the
 * channels (h, d) as output features and the sequence as input features this is Eq. 1 once per
 * head, and the tensor-core kernel runs all heads in one launch (head h = 128-row tile h).
 * Head dimension D = 128; S % 128 == 0.
 *
 * w4a8_pack_value: V_f16 [S][H][D] binary16 (the value projection's output, token-major) ->
 *   blob of w4a8_packed_bytes(H * D, S, 0) bytes (Eq. 5 per channel over the S positions).
 * w4a8_attn_pv: Pq [H][T][S] INT8 and p_scale [H][T] FP32 as written by w4a8_quantize_act on
 *   the attention map viewed as [H * T][S]; O_bf16 [T][H][D] bfloat16:
 *   o = (float(sum_s Pq * t2(code)) * p_scale[h][t]) * (0.5 * step[h][d]).
 *   workspace >= w4a8_attn_pv_workspace_bytes(T, S, H, D), zero-filled once. */
w4a8_status w4a8_pack_value(const void *V_f16, int S, int H, int D, float clip, void *packed,
                            size_t packed_bytes, void *stream);
size_t w4a8_attn_pv_workspace_bytes(int T, int S, int H, int D);
w4a8_status w4a8_attn_pv(const int8_t *Pq, const float *p_scale, const void *packed, int T, int S,
                         int H, int D, void *O_bf16, void *workspace, size_t workspace_bytes,
                         void *stream);

/* w4a8_linear_asym for any group_size: with group_size 128 the token's zero-point leaves every
 * group's integer sum before that sum is scaled,
 *   acc_g[m][n] = sum_{k in g} Xq[m][k] * t2(code[n][k]) - tok_zero[m] * rowsum[g][n],
 *   y = (sum_g float(acc_g) * (0.5 * step[g][n])) * tok_scale[m] + bias[n],
 * rowsum [G][N] as written by w4a8_weight_rowsum with the same group_size; acc, if given, is
 * [G][M][N].  (The paper's W4A8 uses per-channel steps; its group-128 results are weight-only.) */
w4a8_status w4a8_linear_asym_group(const int8_t *Xq, const float *tok_scale, const int32_t *tok_zero,
                                   const void *packed, const int32_t *rowsum, const float *bias,
                                   int M, int N, int K, int group_size, void *Y_bf16, int32_t *acc,
                                   void *workspace, size_t workspace_bytes, void *stream,
                                   const w4a8_opts *opts);

/* Test export: the INT32 accumulators of the contraction, acc [G][M][N], before any
 * rescale (Eq. 6 in units of step/2).  Uses the same kernels as w4a8_linear_ex. */
w4a8_status w4a8_linear_acc_i32(const int8_t *Xq, const void *packed, int M, int N, int K,
                                int group_size, int32_t *acc, void *workspace,
                                size_t workspace_bytes, void *stream,
                                const w4a8_opts *opts);

/* Test export: undo the tiling.  codes [N][K/2] with byte k/2 = code[k] | code[k+1] << 4,
 * scales [G][N] FP32, zeros [G][N] u8. */
w4a8_status w4a8_unpack_codes(const void *packed, int N, int K, int group_size,
                              uint8_t *codes, float *scales, uint8_t *zeros, void *stream);

/* w4a8_unpack_codes for a blob of `bits`-bit codes (3 or 4); codes come two per byte either way
 * (a 3-bit code in the low bits of its nibble). */
w4a8_status w4a8_unpack_codes_bits(const void *packed, int N, int K, int group_size, int bits,
                                   uint8_t *codes, float *scales, uint8_t *zeros, void *stream);

/* Synchronizes `stream`, then reads and clears the status block of `workspace`:
 * W4A8_OK, W4A8_ERR_TIMEOUT or W4A8_ERR_BAD_BLOB (first failure since the last poll).
 * A kernel that gave up (W4A8_ERR_TIMEOUT) may leave split-K tile counters behind in the
 * workspace: run w4a8_workspace_init on it before the next call, else a later split-K call can
 * reduce partial tiles too early.  The output of a call that reported a failure is undefined. */
w4a8_status w4a8_poll_status(void *workspace, void *stream);

/* Host: Eq. 6 in units of step/2 for zero-point z: out[code] = 2 (code - z) for
 * code <= 13, +1 for 14, -1 for 15.  `out` is a host array of 16. */
void w4a8_dint4_table(int z, int8_t *out);

/* Host: the same table in units of step / 2^level_shift: 2^level_shift (code - z), +1, -1. */
void w4a8_dint4_table_fmt(int z, int level_shift, int8_t *out);

/* Host: the table for `bits`-bit codes (3 or 4): 2^level_shift (code - z) for the integer codes
 * 0..p, +1 for code p + 1, -1 for code p + 2; entries past 2^bits are zero.  `out` holds 16. */
void w4a8_dint_table_bits(int z, int bits, int level_shift, int8_t *out);

/* Host: version string with static storage. */
const char *w4a8_version(void);

#ifdef __cplusplus
}
#endif
#endif /* W4A8_H_ */
