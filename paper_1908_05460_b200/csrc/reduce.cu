// Fixed-order sum of split partial results:  dw[i] = alpha * sum_{sp} partial[sp][i], i < count.
// partial is [splits][count] in the element order of dw.  A block handles 32 columns (float4 columns
// when count is a multiple of four); each of its W warps (W = splits rounded up to a power of two, at
// most 32) sums an interleaved subset of the splits in ascending order, and warp 0 adds the W
// subtotals in warp order, so the result does not depend on scheduling.
#include "gaconv_internal.h"

namespace gaconv {
namespace {

constexpr int kReduceWarps = 32;

template <typename V> __device__ __forceinline__ V vzero();
template <> __device__ __forceinline__ float vzero<float>() { return 0.f; }
template <> __device__ __forceinline__ float4 vzero<float4>() { return make_float4(0.f, 0.f, 0.f, 0.f); }
__device__ __forceinline__ void vadd(float& a, const float b) { a += b; }
__device__ __forceinline__ void vadd(float4& a, const float4 b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }
__device__ __forceinline__ float vscale(float a, float s) { return a * s; }
__device__ __forceinline__ float4 vscale(float4 a, float s) { return make_float4(a.x * s, a.y * s, a.z * s, a.w * s); }

template <typename V>
__global__ void __launch_bounds__(32 * kReduceWarps)
reduce_splits_kernel(const V* __restrict__ partial, V* __restrict__ dw, size_t count, int splits, float alpha)
{
    __shared__ V sm[kReduceWarps][32];
    // no early release here: the kernels that follow are sized as one wave, and placing their CTAs while
    // this kernel's large blocks still hold some SMs unbalances that wave
    pdl_wait_prior_grid();
    const int lane = threadIdx.x & 31, grp = threadIdx.x >> 5, warps = blockDim.x >> 5;
    const size_t i = (size_t)blockIdx.x * 32 + lane;
    V acc = vzero<V>();
    if (i < count) {
        const V* p = partial + i;
#pragma unroll 5
        for (int sp = grp; sp < splits; sp += warps) vadd(acc, __ldcg(p + (size_t)sp * count));
    }
    sm[grp][lane] = acc;
    __syncthreads();
    if (grp == 0 && i < count) {
        V t = sm[0][lane];
        const int used = splits < warps ? splits : warps;
        for (int w = 1; w < used; ++w) vadd(t, sm[w][lane]);
        dw[i] = vscale(t, alpha);
    }
}

// Many splits of a small block (hundreds of 9 KB slots after a small layer): 8 float4 columns per block and
// 32 split lanes, so that the work spreads over more SMs and every thread has all its loads in flight
// at once.  Lane l sums splits l, l+32, ... in ascending order; lane 0 of a column adds the 32 subtotals in
// lane order.
__global__ void __launch_bounds__(256)
reduce_splits_many_kernel(const float4* __restrict__ partial, float4* __restrict__ dw, size_t count, int splits, float alpha)
{
    __shared__ float4 sm[32][8];
    pdl_wait_prior_grid();
    const int cq = threadIdx.x & 7, sl = threadIdx.x >> 3;
    const size_t i = (size_t)blockIdx.x * 8 + cq;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < count) {
        const float4* p = partial + i;
#pragma unroll 8
        for (int sp = sl; sp < splits; sp += 32) vadd(acc, __ldcg(p + (size_t)sp * count));
    }
    sm[sl][cq] = acc;
    __syncthreads();
    if (sl == 0 && i < count) {
        float4 t = sm[0][cq];
        const int used = splits < 32 ? splits : 32;
        for (int w = 1; w < used; ++w) vadd(t, sm[w][cq]);
        dw[i] = vscale(t, alpha);
    }
}

}  // namespace

cudaError_t reduce_splits(const float* partial, float* dw, size_t count, int splits, float alpha, cudaStream_t stream)
{
    // as many warps per block as there are splits to share out (a power of two, at most 32)
    int warps = 1;
    while (warps < splits && warps < kReduceWarps) warps *= 2;
    note_launch();
    if (count % 4 == 0 && splits >= 64 && count / 4 <= 65536) {
        const size_t c4 = count / 4;
        return launch_kernel(reduce_splits_many_kernel, dim3((unsigned)((c4 + 7) / 8)), dim3(256), 0, stream, dim3(1, 1, 1),
                             reinterpret_cast<const float4*>(partial), reinterpret_cast<float4*>(dw), c4, splits, alpha);
    }
    if (count % 4 == 0) {
        const size_t c4 = count / 4;
        return launch_kernel(reduce_splits_kernel<float4>, dim3((unsigned)((c4 + 31) / 32)), dim3(32 * warps), 0, stream, dim3(1, 1, 1),
                             reinterpret_cast<const float4*>(partial), reinterpret_cast<float4*>(dw), c4, splits, alpha);
    }
    return launch_kernel(reduce_splits_kernel<float>, dim3((unsigned)((count + 31) / 32)), dim3(32 * warps), 0, stream, dim3(1, 1, 1),
                         partial, dw, count, splits, alpha);
}

}  // namespace gaconv
