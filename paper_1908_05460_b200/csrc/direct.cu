// Exact filter gradient on the FP32 pipes (paper Section 2.4: "to compute df we have to convolve I
// with dO"):   dW[k,c,r,s] = alpha * sum_{n,p,q} Xz[n,c,p*st+r-pad,q*st+s-pad] * dY[n,k,p,q].
// Works for every shape, layout and dtype: products and sums are fp32, so fp32 inputs meet the
// fp32 tolerance class.  It is the anchor the tensor-core path is checked against on shapes the
// oracle cannot cover in full, and the route for shapes the tensor-core path does not tile.
//
// Tiled kernel: a CTA owns a 16 (k) x 16 (c) x R x S block of dW and a range of work items; a work
// item is one image's band of BP x BQ output pixels.  Per item the dY band and the X window are
// staged in shared memory as fp32; thread (tk, tc) keeps its R*S accumulators in registers.
// Splits of the reduction are combined by the last CTA to finish, in split order.
#include "gaconv_internal.h"

namespace gaconv {
namespace {

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) {
    return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
}

constexpr int TK = 16, TC = 16;

template <typename T, int R, int S>
__global__ void __launch_bounds__(256)
direct_tiled_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ dw,
                    float* __restrict__ partial, uint32_t* __restrict__ counters, Geom g, DirectPlan pl)
{
    extern __shared__ float smem[];
    const int win_h = (pl.bp - 1) * g.stride_h + R, win_w = (pl.bq - 1) * g.stride_w + S;
    float* s_dy = smem;                                  // [TK][bp*bq]
    float* s_x = smem + TK * pl.bp * pl.bq;              // [win_h][win_w][TC]
    __shared__ bool s_last;

    const int tile = blockIdx.x, split = blockIdx.y;
    const int k0 = (tile / pl.tiles_c) * TK, c0 = (tile % pl.tiles_c) * TC;
    const int tk = threadIdx.x / TC, tc = threadIdx.x % TC;

    float acc[R * S];
#pragma unroll
    for (int i = 0; i < R * S; ++i) acc[i] = 0.f;

    const int per = (pl.items + pl.splits - 1) / pl.splits;
    const int it_end = min(pl.items, (split + 1) * per);
    for (int it = split * per; it < it_end; ++it) {
        const int n = it / (pl.bands_p * pl.bands_q);
        const int band = it % (pl.bands_p * pl.bands_q);
        const int p0 = (band / pl.bands_q) * pl.bp, q0 = (band % pl.bands_q) * pl.bq;
        __syncthreads();
        for (int i = threadIdx.x; i < TK * pl.bp * pl.bq; i += blockDim.x) {
            const int kk = i / (pl.bp * pl.bq), j = i % (pl.bp * pl.bq);
            const int p = p0 + j / pl.bq, q = q0 + j % pl.bq, k = k0 + kk;
            float v = 0.f;
            if (k < g.k && p < g.p && q < g.q) v = ldf(dy + (((long long)n * g.k + k) * g.p + p) * g.q + q);
            s_dy[i] = v;
        }
        const int h0 = p0 * g.stride_h - g.pad_h, w0 = q0 * g.stride_w - g.pad_w;
        for (int i = threadIdx.x; i < win_h * win_w * TC; i += blockDim.x) {
            const int cc = i % TC, pix = i / TC;
            const int hh = h0 + pix / win_w, ww = w0 + pix % win_w, c = c0 + cc;
            float v = 0.f;
            if (c < g.c && hh >= 0 && hh < g.h && ww >= 0 && ww < g.w)
                v = ldf(x + n * g.xs_n + c * g.xs_c + hh * g.xs_h + ww * g.xs_w);
            s_x[i] = v;
        }
        __syncthreads();
        for (int pp = 0; pp < pl.bp; ++pp)
            for (int qq = 0; qq < pl.bq; ++qq) {
                const float d = s_dy[(tk * pl.bp + pp) * pl.bq + qq];
                const float* xb = s_x + ((pp * g.stride_h) * win_w + qq * g.stride_w) * TC + tc;
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int s = 0; s < S; ++s) acc[r * S + s] = fmaf(d, xb[(r * win_w + s) * TC], acc[r * S + s]);
            }
    }

    const int k = k0 + tk, c = c0 + tc;
    const bool valid = k < g.k && c < g.c;
    if (pl.splits == 1) {
        if (valid)
#pragma unroll
            for (int i = 0; i < R * S; ++i) dw[k * g.ws_k + c * g.ws_c + (i / S) * g.ws_r + (i % S) * g.ws_s] = g.alpha * acc[i];
        return;
    }
    // partial[split][tile][rs][thread]
    const size_t tile_elems = (size_t)R * S * 256;
    float* mine = partial + ((size_t)split * gridDim.x + tile) * tile_elems;
#pragma unroll
    for (int i = 0; i < R * S; ++i) mine[i * 256 + threadIdx.x] = acc[i];
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(&counters[tile % kWsNumCounters], 1u) == (uint32_t)pl.splits - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
#pragma unroll
    for (int i = 0; i < R * S; ++i) {
        float tot = 0.f;
        for (int sp = 0; sp < pl.splits; ++sp)
            tot += __ldcg(partial + ((size_t)sp * gridDim.x + tile) * tile_elems + i * 256 + threadIdx.x);
        if (valid) dw[k * g.ws_k + c * g.ws_c + (i / S) * g.ws_r + (i % S) * g.ws_s] = g.alpha * tot;
    }
    if (threadIdx.x == 0) counters[tile % kWsNumCounters] = 0;
}

// Any filter size: one thread per dW element, whole reduction in the thread.
template <typename T>
__global__ void __launch_bounds__(256)
direct_element_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ dw, Geom g)
{
    const long long total = (long long)g.k * g.r * g.s * g.c;
    const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= total) return;
    const int c = (int)(e % g.c); long long t = e / g.c;
    const int s = (int)(t % g.s); t /= g.s;
    const int r = (int)(t % g.r); const int k = (int)(t / g.r);
    float acc = 0.f;
    for (int n = 0; n < g.n; ++n)
        for (int p = 0; p < g.p; ++p) {
            const int hh = p * g.stride_h + r - g.pad_h;
            if (hh < 0 || hh >= g.h) continue;
            for (int q = 0; q < g.q; ++q) {
                const int ww = q * g.stride_w + s - g.pad_w;
                if (ww < 0 || ww >= g.w) continue;
                acc = fmaf(ldf(x + n * g.xs_n + c * g.xs_c + hh * g.xs_h + ww * g.xs_w),
                           ldf(dy + (((long long)n * g.k + k) * g.p + p) * g.q + q), acc);
            }
        }
    dw[k * g.ws_k + c * g.ws_c + r * g.ws_r + s * g.ws_s] = g.alpha * acc;
}

template <typename T>
cudaError_t launch_t(const T* x, const T* dy, float* dw, float* partial, uint32_t* counters, const Geom& g,
                     const DirectPlan& pl, cudaStream_t stream)
{
    if (!pl.tiled) {
        const long long total = (long long)g.k * g.r * g.s * g.c;
        direct_element_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(x, dy, dw, g);
        note_launch();
        return cudaGetLastError();
    }
    const int win_h = (pl.bp - 1) * g.stride_h + g.r, win_w = (pl.bq - 1) * g.stride_w + g.s;
    const size_t smem = sizeof(float) * ((size_t)TK * pl.bp * pl.bq + (size_t)win_h * win_w * TC);
    dim3 grid(pl.tiles_k * pl.tiles_c, pl.splits);
#define GACONV_DIRECT_CASE(RR, SS)                                                                         \
    if (g.r == RR && g.s == SS) {                                                                          \
        direct_tiled_kernel<T, RR, SS><<<grid, 256, smem, stream>>>(x, dy, dw, partial, counters, g, pl); \
        note_launch();                                                                                     \
        return cudaGetLastError();                                                                         \
    }
    GACONV_DIRECT_CASE(1, 1)
    GACONV_DIRECT_CASE(3, 3)
    GACONV_DIRECT_CASE(5, 5)
#undef GACONV_DIRECT_CASE
    return cudaErrorInvalidValue;
}

}  // namespace

DirectPlan plan_direct(const Geom& g)
{
    DirectPlan pl{};
    pl.tiled = (g.r == g.s) && (g.r == 1 || g.r == 3 || g.r == 5);
    pl.tiles_k = (g.k + TK - 1) / TK;
    pl.tiles_c = (g.c + TC - 1) / TC;
    pl.bq = g.q < 32 ? g.q : 32;
    pl.bp = g.p < 4 ? g.p : 4;
    while (pl.bp * 2 <= g.p && pl.bp * pl.bq < 128) pl.bp *= 2;
    // shared memory must stay under the default 48 KiB
    auto smem = [&](int bp, int bq) {
        return sizeof(float) * ((size_t)TK * bp * bq + (size_t)((bp - 1) * g.stride_h + g.r) * ((bq - 1) * g.stride_w + g.s) * TC);
    };
    while (pl.bp > 1 && smem(pl.bp, pl.bq) > 40 * 1024) pl.bp /= 2;
    while (pl.bq > 1 && smem(pl.bp, pl.bq) > 40 * 1024) pl.bq /= 2;
    pl.bands_p = (g.p + pl.bp - 1) / pl.bp;
    pl.bands_q = (g.q + pl.bq - 1) / pl.bq;
    pl.items = g.n * pl.bands_p * pl.bands_q;
    const int tiles = pl.tiles_k * pl.tiles_c;
    int splits = (148 * 4 + tiles - 1) / tiles;
    if (splits > pl.items) splits = pl.items;
    if (tiles > kWsNumCounters) splits = 1;
    const size_t tile_bytes = (size_t)g.r * g.s * 256 * sizeof(float);
    while (splits > 1 && (size_t)splits * tiles * tile_bytes > ((size_t)64 << 20)) --splits;
    if (splits < 1) splits = 1;
    if (!pl.tiled) splits = 1;
    pl.splits = splits;
    pl.partial_bytes = splits > 1 ? (size_t)splits * tiles * tile_bytes : 0;
    return pl;
}

cudaError_t launch_direct(const void* x, const void* dy, float* dw, float* partial, uint32_t* counters,
                          const Geom& g, const DirectPlan& plan, cudaStream_t stream)
{
    if (g.bf16)
        return launch_t(static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(dy), dw, partial,
                        counters, g, plan, stream);
    return launch_t(static_cast<const float*>(x), static_cast<const float*>(dy), dw, partial, counters, g, plan, stream);
}

}  // namespace gaconv
