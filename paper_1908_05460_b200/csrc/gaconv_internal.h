// Internal declarations shared by the translation units of libgaconv (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

#include "gaconv.h"

#include <utility>

namespace gaconv {

// ---- workspace layout -------------------------------------------------------------------------
// [0, 256)            control: word 0 = sticky device status (0 ok, 1 bounded wait gave up)
// [256, 256+16 KiB)   ticket counters, all zero between calls (each kernel resets what it used)
// [kWsDataOffset, ..) per-call data (selection results, split partials)
constexpr size_t kWsCounterOffset = 256;
constexpr int    kWsNumCounters   = 4096;
constexpr size_t kWsDataOffset    = kWsCounterOffset + sizeof(uint32_t) * kWsNumCounters;

void note_launch(int count = 1);   // bookkeeping behind gaconv_launch_count()

// ---- programmatic dependent launch ------------------------------------------------------------
// Every kernel of the library is launched with programmatic stream serialization allowed and starts
// with pdl_release_next_grid(): the next kernel in the stream may then be scheduled while this one is
// still running, and do its own set-up (barrier init, tensor-memory allocation) early.  Before its
// first access to global memory every kernel executes pdl_wait_prior_grid(), which returns only when
// the previous kernel has completed and its writes are visible -- so results never depend on it.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_release_next_grid() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_prior_grid() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 dim3 cluster, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int n = 0;
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (cluster.x * cluster.y * cluster.z > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = cluster.x; attr[n].val.clusterDim.y = cluster.y; attr[n].val.clusterDim.z = cluster.z;
        ++n;
    }
    cfg.attrs = attr; cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Geometry with derived sizes and element strides of the chosen layouts.
struct Geom {
    int n, c, h, w, k, r, s, p, q;
    int stride_h, stride_w, pad_h, pad_w;
    long long xs_n, xs_c, xs_h, xs_w;   // element strides of X
    long long ws_k, ws_c, ws_r, ws_s;   // element strides of dW
    bool bf16;
    float alpha;
    int sm_budget;                      // 0: plan for the whole GPU; n > 0: for about n SMs
};

// ---- out[b][j][i] = in[b][i][j], i < rows, j < cols: N x C x H x W activations -> N x H x W x C, N x P x Q x K gradients -> N x K x P x Q ----
cudaError_t launch_transpose_batched(const void* in, void* out, int rows, int cols, int batch, bool bf16, cudaStream_t stream);

// ---- fixed-order sum of split partials: dw = alpha * sum_sp partial[sp][0..count) ----
cudaError_t reduce_splits(const float* partial, float* dw, size_t count, int splits, float alpha, cudaStream_t stream);

// ---- selection (Algorithm 1, arg-max and sum lines) ----
cudaError_t launch_select(const void* dy, int32_t* idx, float* sum, void* dy_sparse, const Geom& g,
                          cudaStream_t stream);

// selection written as the transposed sparse tensor dYt'[n][j][k] (bf16, maps of fewer than 64 pixels, k % 8 == 0)
cudaError_t launch_select_sparse_transposed(const void* dy, void* dyt, const Geom& g, cudaStream_t stream);

// ---- gather-accumulate (Algorithm 1, patch accumulation line) ----
struct GatherPlan {
    int chunks;          // CTAs per output channel, each owning a contiguous range of images
    int imgs_per_chunk;
    size_t partial_bytes;
};
GatherPlan plan_gather(const Geom& g);
cudaError_t launch_gather(const void* x, const int32_t* idx, const float* sum, float* dw, float* partial,
                          uint32_t* counters, const Geom& g, const GatherPlan& plan, int topk, cudaStream_t stream);
// selection of the top-k variant: idx[map][topk] in order of selection, sum[map]
cudaError_t launch_select_topk(const void* dy, int32_t* idx, float* sum, const Geom& g, int topk, cudaStream_t stream);

// ---- Algorithm 1 in one launch (selection + patch accumulate + cluster reduction) ----
bool top1_fused_supported(const Geom& g);
cudaError_t launch_top1_fused(const void* x, const void* dy, float* dw, const Geom& g, cudaStream_t stream,
                              const int32_t* sel_idx = nullptr, const float* sel_sum = nullptr, int topk = 1);

// ---- zero / random gradient ----
cudaError_t launch_zero(float* dw, size_t count, cudaStream_t stream);
cudaError_t launch_random(float* dw, const Geom& g, uint64_t seed, float std, cudaStream_t stream);

// ---- exact filter gradient, direct FP32 kernel (any shape, any layout) ----
struct DirectPlan {
    int tiles_k, tiles_c;   // output tiles of 16 x 16 (k x c), all (r,s) per tile
    int bp, bq;             // output-pixel band handled per work item
    int bands_p, bands_q;
    int items;              // n * bands_p * bands_q
    int splits;             // CTAs per output tile along the reduction
    size_t partial_bytes;
    bool tiled;             // false: filter size without a tiled instantiation -> per-element kernel
    bool vec_dy, vec_x;     // 4-element vector loads usable for the dY band / the X window
};
DirectPlan plan_direct(const Geom& g);
cudaError_t launch_direct(const void* x, const void* dy, float* dw, float* partial, uint32_t* status,
                          const Geom& g, const DirectPlan& plan, cudaStream_t stream);

// ---- exact filter gradient, fp32 inputs on mma.sync with split TF32 operands (3 passes: fp32 accuracy) ----
bool direct_mma_supported(const Geom& g, const DirectPlan& plan);
cudaError_t launch_direct_mma(const void* x, const void* dy, float* dw, float* partial, uint32_t* status, const Geom& g,
                              const DirectPlan& plan, bool three_pass, cudaStream_t stream);

// ---- exact filter gradient for layers with at most four input channels (stems), mma.sync over flattened image rows ----
struct StemPlan {
    size_t partial_bytes;
    alignas(8) unsigned char opaque[256];   // kernel parameters, private to stem_mma.cu
};
bool plan_stem(const Geom& g, StemPlan* plan);
cudaError_t launch_stem(const void* x, const void* dy, float* dw, float* partial, uint32_t* status, const StemPlan& plan,
                        cudaStream_t stream);

// ---- exact filter gradient on tcgen05 tensor cores (bf16, NHWC X, shapes its tiling covers) ----
struct TcPlan {
    size_t partial_bytes;
    size_t scratch_bytes;                   // extra device scratch (transposed dY for very small maps)
    bool reads_transposed_dy;               // the kernel's dY operand is the transposed copy dYt[n][pq][k] in the scratch
    bool stacked_rows;                      // the filter rows share one MMA (stacked in M): few output channels, "same" padding
    alignas(8) unsigned char opaque[512];   // kernel parameters, private to tc.cu
};
bool plan_tc(const Geom& g, TcPlan* plan);   // false: shape not covered, use the direct kernel
// fp32 inputs on the same kernel with TF32 MMAs: passes = 3 (split operands, fp32 accuracy) or 1 (plain TF32)
bool plan_tc_f32(const Geom& g, int passes, TcPlan* plan);
// dy == nullptr: the scratch already holds the transposed operand (plan.reads_transposed_dy only)
cudaError_t launch_tc(const void* x, const void* dy, float* dw, float* partial, void* scratch, uint32_t* counters,
                      uint32_t* status,
                      const TcPlan& plan, cudaStream_t stream);

}  // namespace gaconv
