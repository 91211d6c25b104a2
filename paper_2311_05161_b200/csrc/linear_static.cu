// w4a8_linear_static: the quantized linear layer for callers that cannot hand over a
// workspace.  The scratch the tensor-core kernel needs (status block, split-K tile
// counters, split-K partial tiles) lives in a fixed device array that is part of the
// library image, so this entry point allocates nothing, neither directly nor through a
// library routine.
#include <mutex>

#include "common.cuh"

namespace {

// Every device that loads the library holds this array until the process exits.
constexpr size_t kStaticScratchBytes = (size_t)8 << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
unsigned char *g_scratch_addr[kMaxDevices] = {};

// Device address of the array on the current device.  In host code the symbol
// g_static_scratch is only a handle, so the address is asked for once per device, with that
// device current, and remembered.
w4a8_status scratch_for_current_device(unsigned char **out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return W4A8_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return W4A8_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return W4A8_ERR_CUDA;
        g_scratch_addr[dev] = static_cast<unsigned char *>(p);
    }
    *out = g_scratch_addr[dev];
    return W4A8_OK;
}

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

extern "C" w4a8_status w4a8_linear_static(const int8_t *Xq, const float *tok_scale,
                                          const void *packed, const float *bias, int M, int N,
                                          int K, int group_size, void *Y_bf16, void *stream)
{
    using namespace w4a8;
    if (!Xq || !tok_scale || !packed || !Y_bf16) return W4A8_ERR_NULL;
    if (!shape_ok(N, K, group_size) || M < 1) return W4A8_ERR_SHAPE;
    if (!aligned(Xq, 16) || !aligned(tok_scale, 4) || !aligned(bias, 4) || !aligned(Y_bf16, 16) ||
        !aligned(packed, 256))
        return W4A8_ERR_ALIGN;
    const BlobLayout L = make_layout(N, K, group_size);
    LinearPlan plan;
    if (!make_plan(M, L, nullptr, &plan)) return W4A8_ERR_SHAPE;
    if (plan.workspace_bytes > kStaticScratchBytes) return W4A8_ERR_BUFFER_TOO_SMALL;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return W4A8_ERR_CUDA;
    if (major != 10) return W4A8_ERR_UNSUPPORTED_ARCH;
    unsigned char *scratch = nullptr;
    const w4a8_status s = scratch_for_current_device(&scratch);
    if (s != W4A8_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array keeps whatever the previous call left: the status block and the tile
    // counters must start at zero (the partial tiles are fully written before they are read).
    if (cudaMemsetAsync(scratch, 0, plan.off_partials, st) != cudaSuccess) return W4A8_ERR_CUDA;
    return launch_linear_tcgen05(Xq, tok_scale, static_cast<const uint8_t *>(packed), L, bias, M,
                                 static_cast<__nv_bfloat16 *>(Y_bf16), nullptr, scratch, plan, st);
}

// What the kernel of the last w4a8_linear_static call on this device reported: the status block
// at the head of the array, read after `stream` has drained (the next call clears it).  Copies
// twelve bytes to the host; allocates nothing.
extern "C" w4a8_status w4a8_static_poll_status(void *stream)
{
    unsigned char *scratch = nullptr;
    const w4a8_status s = scratch_for_current_device(&scratch);
    if (s != W4A8_OK) return s;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return W4A8_ERR_CUDA;
    int host[3] = {0, 0, 0};
    if (cudaMemcpy(host, scratch, sizeof(host), cudaMemcpyDeviceToHost) != cudaSuccess) return W4A8_ERR_CUDA;
    if (host[0] == 0) return W4A8_OK;
    return host[0] == W4A8_ERR_BAD_BLOB ? W4A8_ERR_BAD_BLOB : W4A8_ERR_TIMEOUT;
}
