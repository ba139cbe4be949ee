// Operands given in the other order are brought into the kernels' own by one pass through shared memory into the
// caller's workspace: activations N x C x H x W -> N x H x W x C (what the tensor-core, stem and gather kernels are
// built for), output gradients N x P x Q x K -> N x K x P x Q.  (The paper's own kernel expects channels-last
// activations as well and pays the same transposition, Sections 2.4 and 3.1.)
#include "gaconv_internal.h"

namespace gaconv {
namespace {

// out[b][j][i] = in[b][i][j] for i < c, j < hw.  A block turns a 32 x 32 tile; both the reads (along j) and the
// writes (along i) are contiguous.
template <typename T>
__global__ void __launch_bounds__(256)
transpose_batched_kernel(const T* __restrict__ in, T* __restrict__ out, int c, int hw)
{
    __shared__ T tile[32][33];
    pdl_release_next_grid();
    pdl_wait_prior_grid();
    const int n = blockIdx.z, j0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    const T* src = in + (size_t)n * c * hw;
    T* dst = out + (size_t)n * c * hw;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int cc = ty; cc < 32; cc += 8)
        if (c0 + cc < c && j0 + tx < hw) tile[cc][tx] = src[(size_t)(c0 + cc) * hw + j0 + tx];
    __syncthreads();
    for (int jj = ty; jj < 32; jj += 8)
        if (j0 + jj < hw && c0 + tx < c) dst[(size_t)(j0 + jj) * c + c0 + tx] = tile[tx][jj];
}

}  // namespace

cudaError_t launch_transpose_batched(const void* in, void* out, int rows, int cols, int batch, bool bf16, cudaStream_t stream)
{
    const dim3 grid((unsigned)((cols + 31) / 32), (unsigned)((rows + 31) / 32), (unsigned)batch);
    if (grid.y > 65535u || grid.z > 65535u) return cudaErrorInvalidValue;
    note_launch();
    if (bf16)
        return launch_kernel(transpose_batched_kernel<__nv_bfloat16>, grid, dim3(256), 0, stream, dim3(1, 1, 1),
                             static_cast<const __nv_bfloat16*>(in), static_cast<__nv_bfloat16*>(out), rows, cols);
    return launch_kernel(transpose_batched_kernel<float>, grid, dim3(256), 0, stream, dim3(1, 1, 1), static_cast<const float*>(in),
                         static_cast<float*>(out), rows, cols);
}

}  // namespace gaconv
