// gaconv_dw_exact_static: the exact filter gradient for callers that cannot allocate device memory.
//
// Some callers have no way to hand the library a workspace: code running where cudaMalloc is off
// limits -- inside a region that must not touch the allocator (a latency-critical loop that was
// promised "no allocation after warm-up", a plugin that only receives its inputs and outputs from a
// host framework, a process whose memory pool is owned by someone else).  For them this entry point
// keeps the scratch the exact path needs (split partial sums and the control words) in a fixed
// array that is part of the library image: every GPU that loads the library holds
// kStaticScratchBytes of it until the process exits.
//
// The array's name is only a host-side handle: its device address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and that address is what the kernels receive.
#include <mutex>

#include "gaconv_internal.h"

namespace {

constexpr size_t kStaticScratchBytes = (size_t)8 << 20;     // 8 MiB per GPU that loads the library
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};                        // device address of the array, per device

// First call on a device: resolve the array's device address and zero its control words (the rest
// needs no initial value: every call overwrites the partial sums it later reads).
gaconv_status_t static_scratch_for_current_device(cudaStream_t stream, void** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return GACONV_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return GACONV_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_ptr[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return GACONV_ERR_CUDA;
        if (cudaMemsetAsync(ptr, 0, gaconv::kWsDataOffset, stream) != cudaSuccess) return GACONV_ERR_CUDA;
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return GACONV_OK;
}

}  // namespace

extern "C" {

size_t gaconv_static_scratch_bytes(void) { return kStaticScratchBytes; }

// The status word of the built-in array (its first four bytes) is where a kernel launched through
// gaconv_dw_exact_static records that it gave up on a bounded wait.  Read and cleared like the
// caller-owned workspace's word; no allocation, and nothing to do before the array's first use.
gaconv_status_t gaconv_poll_async_status_static(void* stream)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return GACONV_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return GACONV_ERR_UNSUPPORTED;
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        scratch = g_scratch_ptr[dev];
    }
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (scratch == nullptr) return cudaStreamSynchronize(cs) == cudaSuccess ? GACONV_OK : GACONV_ERR_CUDA;
    uint32_t word = 0;
    if (cudaMemcpyAsync(&word, scratch, sizeof(word), cudaMemcpyDeviceToHost, cs) != cudaSuccess) return GACONV_ERR_CUDA;
    if (cudaStreamSynchronize(cs) != cudaSuccess) return GACONV_ERR_CUDA;
    if (word == 0) return GACONV_OK;
    if (cudaMemsetAsync(scratch, 0, sizeof(word), cs) != cudaSuccess) return GACONV_ERR_CUDA;
    return GACONV_ERR_TIMEOUT;
}

gaconv_status_t gaconv_dw_exact_static(const void* x, const void* dy, float* dw, const gaconv_conv_desc_t* desc, void* stream)
{
    if (desc == nullptr) return GACONV_ERR_NULL_POINTER;
    size_t need = 0;
    gaconv_status_t st = gaconv_workspace_size(desc, GACONV_METHOD_EXACT, &need);
    if (st != GACONV_OK) return st;
    if (need > kStaticScratchBytes) return GACONV_ERR_WORKSPACE_TOO_SMALL;   // problem too large for the built-in scratch
    if (x == nullptr || dy == nullptr || dw == nullptr) return GACONV_ERR_NULL_POINTER;
    void* scratch = nullptr;
    st = static_scratch_for_current_device(static_cast<cudaStream_t>(stream), &scratch);
    if (st != GACONV_OK) return st;
    gaconv_conv_desc_t local = *desc;          // same problem, scratch replaced by the built-in array
    local.workspace = scratch;
    local.workspace_bytes = kStaticScratchBytes;
    return gaconv_dw_exact(x, dy, dw, &local, stream);
}

}  // extern "C"
