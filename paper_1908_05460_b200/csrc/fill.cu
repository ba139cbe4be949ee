// Zero gradient (paper Section 2.1) and random gradient (Section 2.2).
//
// Random gradient: independent N(0, std^2) values from a counter-based generator, so that a value
// depends only on (seed, element index) and a new seed per batch regenerates everything:
//   Philox-4x32-10 (Salmon et al., SC'11), key = (seed low, seed high), counter = (j,0,0,0)
//   -> words w0..w3 -> elements 4j..4j+3 by Box-Muller:
//   u1 = (w_a+1) 2^-32, u2 = w_b 2^-32, rho = sqrt(-2 ln u1), (rho cos 2 pi u2, rho sin 2 pi u2)
// for the pairs (w0,w1) and (w2,w3).  Element i is position i of the logical [k][c][r][s] order.
#include "gaconv_internal.h"

namespace gaconv {
namespace {

__global__ void __launch_bounds__(256) zero_kernel(float* __restrict__ dw, size_t count)
{
    pdl_release_next_grid();
    pdl_wait_prior_grid();
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t nvec = count / 4;
    float4* v = reinterpret_cast<float4*>(dw);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += stride)
        v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (size_t i = nvec * 4 + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += stride) dw[i] = 0.f;
}

__device__ __forceinline__ void philox_round(uint32_t (&c)[4], uint32_t k0, uint32_t k1)
{
    const uint32_t hi0 = __umulhi(0xD2511F53u, c[0]), lo0 = 0xD2511F53u * c[0];
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c[2]), lo1 = 0xCD9E8D57u * c[2];
    const uint32_t n0 = hi1 ^ c[1] ^ k0, n2 = hi0 ^ c[3] ^ k1;
    c[0] = n0; c[1] = lo1; c[2] = n2; c[3] = lo0;
}

// Box-Muller on the special-function unit.  The result has to be within 1e-5 * max(1, |z|) of the real-number
// value of the formula, which leaves room for the fast approximations as long as no argument is rounded where
// rounding is amplified:
//   ln u1   u1 = (wa+1) 2^-32.  Away from 1 the hardware logarithm of the rounded value is accurate to ~2^-21
//           in absolute terms; for u1 > 1 - 2^-7 the logarithm is small and that is not enough, but there
//           1-u1 = t 2^-32 with t an integer below 2^25 (exact in fp32 up to rounding of 2^-24 relative) and
//           ln(1-f) = -(f + f^2/2 + f^3/3 + f^4/4) is accurate to f^5/5 < 2^-37.
//   angle   2 pi u2 with u2 = wb 2^-32: taking wb as a signed integer moves the angle to [-pi, pi), where the
//           hardware sine and cosine have their stated absolute accuracy (2^-21.4), without changing the value.
__device__ __forceinline__ void box_muller(uint32_t wa, uint32_t wb, float& z0, float& z1)
{
    const uint32_t t = 0xffffffffu - wa;                          // 2^32 - (wa+1)
    const float f = (float)t * (1.0f / 4294967296.0f);            // 1 - u1
    const float u1 = (wa < 0x7fffffffu) ? (float)(wa + 1u) * (1.0f / 4294967296.0f) : 1.0f - f;
    const float ln_far = __logf(u1);
    const float ln_near = -f * fmaf(f, fmaf(f, fmaf(f, 0.25f, 1.0f / 3.0f), 0.5f), 1.0f);
    const float ln_u1 = (t < (1u << 25)) ? ln_near : ln_far;
    const float rho = __fsqrt_rn(-2.0f * ln_u1);
    const float theta = (float)(int32_t)wb * (6.283185307179586f / 4294967296.0f);
    z0 = rho * __cosf(theta); z1 = rho * __sinf(theta);
}

// philox words of counter j -> four standard normals
__device__ __forceinline__ void normals4(uint32_t j, uint32_t key0, uint32_t key1, float (&z)[4])
{
    uint32_t c[4] = {j, 0u, 0u, 0u};
    uint32_t k0 = key0, k1 = key1;
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        philox_round(c, k0, k1);
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    box_muller(c[0], c[1], z[0], z[1]);
    box_muller(c[2], c[3], z[2], z[3]);
}

// dW stored in the logical [k][c][r][s] order: thread j writes elements 4j..4j+3 as one 16-byte store.
__global__ void __launch_bounds__(256)
random_kcrs_kernel(float* __restrict__ dw, size_t count, uint32_t key0, uint32_t key1, float std)
{
    pdl_release_next_grid();
    const size_t j = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (4 * j >= count) return;
    float z[4];
    normals4((uint32_t)j, key0, key1, z);
    pdl_wait_prior_grid();      // the values need no memory; only the stores wait for the previous kernel
    if (4 * j + 3 < count) {
        reinterpret_cast<float4*>(dw)[j] = make_float4(std * z[0], std * z[1], std * z[2], std * z[3]);
    } else {
        for (int t = 0; 4 * j + t < count; ++t) dw[4 * j + t] = std * z[t];
    }
}

// Any other dW layout.  grid (channel chunks, K): a CTA draws the values of one output channel k and `cc`
// input channels -- a contiguous range of the logical order, so one Philox call still yields four values --
// into shared memory as [c][r*s], then writes them in storage order: for every (r,s) the chunk's channels,
// which in the [k][r][s][c] layout are contiguous (16-byte stores when the chunk allows).
__global__ void __launch_bounds__(256)
random_strided_kernel(float* __restrict__ dw, Geom g, int cc, uint32_t key0, uint32_t key1, float std)
{
    extern __shared__ float vals[];          // [cc][rs]
    pdl_release_next_grid();
    const int rs = g.r * g.s, k = blockIdx.y, c0 = blockIdx.x * cc, cn = min(cc, g.c - c0), len = cn * rs;
    const size_t first = ((size_t)k * g.c + c0) * rs;       // logical index of the chunk's first element
    const size_t j0 = first / 4;
    const int head = (int)(first - 4 * j0);                  // elements of counter j0 that belong to the previous chunk
    for (int i = threadIdx.x; 4 * i < len + head; i += blockDim.x) {
        float z[4];
        normals4((uint32_t)(j0 + i), key0, key1, z);
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int e = 4 * i + t - head;
            if (e >= 0 && e < len) vals[e] = std * z[t];
        }
    }
    __syncthreads();
    pdl_wait_prior_grid();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
    const bool vec = g.ws_c == 1 && (cn & 3) == 0 && (c0 & 3) == 0 && ((g.ws_k | g.ws_r | g.ws_s) & 3) == 0;
    for (int p = warp; p < rs; p += warps) {
        const int r = p / g.s, s = p - r * g.s;
        float* row = dw + (size_t)k * g.ws_k + (size_t)r * g.ws_r + (size_t)s * g.ws_s + (size_t)c0 * g.ws_c;
        if (vec) {
            for (int c = 4 * lane; c < cn; c += 128)
                *reinterpret_cast<float4*>(row + c) = make_float4(vals[c * rs + p], vals[(c + 1) * rs + p], vals[(c + 2) * rs + p], vals[(c + 3) * rs + p]);
        } else {
            for (int c = lane; c < cn; c += 32) row[(size_t)c * g.ws_c] = vals[c * rs + p];
        }
    }
}

}  // namespace

cudaError_t launch_zero(float* dw, size_t count, cudaStream_t stream)
{
    size_t blocks = (count / 4 + 255) / 256;
    if (blocks < 1) blocks = 1;
    if (blocks > 148 * 8) blocks = 148 * 8;
    note_launch();
    return launch_kernel(zero_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, dim3(1, 1, 1), dw, count);
}

cudaError_t launch_random(float* dw, const Geom& g, uint64_t seed, float std, cudaStream_t stream)
{
    const size_t count = (size_t)g.k * g.c * g.r * g.s;
    const bool contiguous = (g.ws_s == 1 && g.ws_r == g.s && g.ws_c == (long long)g.r * g.s && g.ws_k == (long long)g.c * g.r * g.s);
    const uint32_t key0 = (uint32_t)seed, key1 = (uint32_t)(seed >> 32);
    note_launch();
    if (contiguous) {
        const size_t threads = (count + 3) / 4;
        return launch_kernel(random_kcrs_kernel, dim3((unsigned)((threads + 255) / 256)), dim3(256), 0, stream, dim3(1, 1, 1), dw, count,
                             key0, key1, std);
    }
    // channels per CTA: at most 32 KiB of values, and enough CTAs for the machine when K is small
    const int rs = g.r * g.s;
    int cc = g.c;
    while (cc > 4 && ((size_t)cc * rs * 4 > 32 * 1024 || (long long)g.k * ((g.c + cc - 1) / cc) < 296)) cc = (cc + 1) / 2;
    cc = (cc + 3) / 4 * 4;
    if ((size_t)cc * rs * 4 > 48 * 1024) cc = 4;
    if ((size_t)cc * rs * 4 > 48 * 1024) return cudaErrorInvalidValue;      // filters of thousands of taps: not a case this library meets
    return launch_kernel(random_strided_kernel, dim3((unsigned)((g.c + cc - 1) / cc), (unsigned)g.k), dim3(256), (size_t)cc * rs * 4, stream,
                         dim3(1, 1, 1), dw, g, cc, key0, key1, std);
}

}  // namespace gaconv
