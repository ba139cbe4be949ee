// Exact filter gradient on the FP32 pipes (paper Section 2.4: "to compute df we have to convolve I
// with dO"):   dW[k,c,r,s] = alpha * sum_{n,p,q} Xz[n,c,p*st+r-pad,q*st+s-pad] * dY[n,k,p,q].
// Works for every shape, layout and dtype: products and sums are fp32, so fp32 inputs meet the
// fp32 tolerance class.  It serves fp32 inputs, the 3-channel stem layers and every shape the
// tensor-core path does not tile.
//
// Register-tiled kernel.  A CTA owns a (TKT*OTK) x (TCT*OTC) block of (k, c) with all R*S filter
// taps, and a contiguous range of work items; an item is one image's band of BP x BQ output pixels.
// Per item the dY band ([k][pixel]) and the X window ([row][col][c]) are staged in shared memory
// as fp32, two stages deep: fp32 inputs are copied with 16-byte cp.async while the previous item is
// being consumed; other inputs are converted on the way in.  The OTK*OTC "output threads" of a pixel
// group each keep TKT*TCT*R*S accumulators in registers; the 128/(OTK*OTC) pixel groups take the
// band's pixels round-robin, so one vector load of dY and R*S vector loads of X feed
// TKT*TCT*R*S FMAs.  At the end the pixel groups are summed (warp shuffles, then shared memory, in a
// fixed order) and the CTA writes its block: to dW if it is the only split, else to its slot of
// the partial buffer, which reduce_splits() adds up in split order.
#include "gaconv_internal.h"

namespace gaconv {
namespace {

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) {
    return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p)) << 16);
}

// four consecutive elements as floats (16-byte load for fp32, 8-byte load for bf16)
__device__ __forceinline__ void ld4(const float* p, float (&v)[4]) {
    const float4 t = __ldg(reinterpret_cast<const float4*>(p));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
__device__ __forceinline__ void ld4(const __nv_bfloat16* p, float (&v)[4]) {
    const uint2 t = __ldg(reinterpret_cast<const uint2*>(p));
    v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
    v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
}

constexpr int kThreads = 128;

template <int N> struct Vec;
template <> struct Vec<1> { float v[1]; __device__ void load(const float* p) { v[0] = *p; } };
template <> struct Vec<2> { float v[2]; __device__ void load(const float* p) { float2 t = *reinterpret_cast<const float2*>(p); v[0] = t.x; v[1] = t.y; } };
template <> struct Vec<4> { float v[4]; __device__ void load(const float* p) { float4 t = *reinterpret_cast<const float4*>(p); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; } };

// 16-byte asynchronous global -> shared copy (fp32 fast path) and its group bookkeeping
__device__ __forceinline__ void cp_async16(float* smem_dst, const float* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Stage one work item: dY band as [k][pixel] (row stride dys) and X window as [row][col][TC], fp32.
// ASYNC (fp32 inputs, vector paths): 16-byte cp.async copies, zeros stored directly where the
// tile leaves the tensor.  Otherwise: synchronous loads with conversion.
template <typename T, bool ASYNC, int TK, int TC>
__device__ __forceinline__ void stage_item(const T* __restrict__ x, const T* __restrict__ dy, float* s_dy, float* s_x,
                                           const Geom& g, const DirectPlan& pl, int it, int k0, int c0, int dys,
                                           int win_h, int win_w)
{
    const int npx = pl.bp * pl.bq;
    const int n = it / (pl.bands_p * pl.bands_q);
    const int band = it % (pl.bands_p * pl.bands_q);
    const int p0 = (band / pl.bands_q) * pl.bp, q0 = (band % pl.bands_q) * pl.bq;
    const int h0 = p0 * g.stride_h - g.pad_h, w0 = q0 * g.stride_w - g.pad_w;
    if (pl.vec_dy) {
        const int quads = npx >> 2;
        for (int i = threadIdx.x; i < TK * quads; i += kThreads) {
            const int kk = i / quads, j = (i - kk * quads) << 2, k = k0 + kk;
            float* dst = s_dy + kk * dys + j;
            const T* src = dy + ((long long)n * g.k + k) * g.p * g.q + (long long)p0 * g.q + j;
            if constexpr (ASYNC) {
                if (k < g.k) cp_async16(dst, reinterpret_cast<const float*>(src));
                else *reinterpret_cast<float4*>(dst) = make_float4(0.f, 0.f, 0.f, 0.f);
            } else {
                float v[4] = {0.f, 0.f, 0.f, 0.f};
                if (k < g.k) ld4(src, v);
                *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
            }
        }
    } else {
        for (int i = threadIdx.x; i < TK * npx; i += kThreads) {
            const int kk = i / npx, j = i % npx;
            const int p = p0 + j / pl.bq, q = q0 + j % pl.bq, k = k0 + kk;
            float v = 0.f;
            if (k < g.k && p < g.p && q < g.q) v = ldf(dy + (((long long)n * g.k + k) * g.p + p) * g.q + q);
            s_dy[kk * dys + j] = v;
        }
    }
    if (pl.vec_x) {
        constexpr int CQ = TC / 4;                                // channel quads per pixel of the tile
        for (int hh = 0; hh < win_h; ++hh) {
            const int h = h0 + hh;
            const bool row_ok = h >= 0 && h < g.h;
            const T* xrow = x + n * g.xs_n + (long long)h * g.xs_h;
            float* drow = s_x + hh * win_w * TC;
            for (int i = threadIdx.x; i < win_w * CQ; i += kThreads) {
                const int wq = i / CQ, cq = i - wq * CQ, ww = w0 + wq, c = c0 + 4 * cq;
                const bool ok = row_ok && ww >= 0 && ww < g.w && c < g.c;
                if constexpr (ASYNC) {
                    if (ok) cp_async16(drow + i * 4, reinterpret_cast<const float*>(xrow + (long long)ww * g.xs_w + c));
                    else *reinterpret_cast<float4*>(drow + i * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
                } else {
                    float v[4] = {0.f, 0.f, 0.f, 0.f};
                    if (ok) ld4(xrow + (long long)ww * g.xs_w + c, v);
                    *reinterpret_cast<float4*>(drow + i * 4) = make_float4(v[0], v[1], v[2], v[3]);
                }
            }
        }
    } else {
        for (int i = threadIdx.x; i < win_h * win_w * TC; i += kThreads) {
            const int cc = i % TC, pix = i / TC;
            const int hh = h0 + pix / win_w, ww = w0 + pix % win_w, c = c0 + cc;
            float v = 0.f;
            if (c < g.c && hh >= 0 && hh < g.h && ww >= 0 && ww < g.w)
                v = ldf(x + n * g.xs_n + c * g.xs_c + hh * g.xs_h + ww * g.xs_w);
            s_x[i] = v;
        }
    }
}

template <typename T, bool ASYNC, int R, int S, int TKT, int TCT, int OTK, int OTC>
__global__ void __launch_bounds__(kThreads)
direct_tiled_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ dw,
                    float* __restrict__ partial, Geom g, DirectPlan pl)
{
    constexpr int TK = TKT * OTK, TC = TCT * OTC, OT = OTK * OTC, PG = kThreads / OT, ACC = TKT * TCT * R * S;
    static_assert(kThreads % OT == 0 && OT <= 64, "output threads must divide the CTA");
    extern __shared__ __align__(16) float smem[];
    const int npx = pl.bp * pl.bq;
    const int dys = npx + 4;                     // row stride of the dY band: keeps rows 16-byte aligned, spreads banks
    const int win_h = (pl.bp - 1) * g.stride_h + R, win_w = (pl.bq - 1) * g.stride_w + S;
    const int stage_floats = TK * dys + win_h * win_w * TC;   // a multiple of four
    // two stages: the next item is fetched while the current one is consumed

    const int tile = blockIdx.x, split = blockIdx.y;
    const int k0 = (tile / pl.tiles_c) * TK, c0 = (tile % pl.tiles_c) * TC;
    const int ot = threadIdx.x % OT, pg = threadIdx.x / OT;
    const int otk = ot / OTC, otc = ot % OTC;

    float acc[ACC];
#pragma unroll
    for (int i = 0; i < ACC; ++i) acc[i] = 0.f;

    const int per = (pl.items + pl.splits - 1) / pl.splits;
    const int it_begin = split * per, it_end = min(pl.items, (split + 1) * per);
    if (it_begin < it_end) {
        stage_item<T, ASYNC, TK, TC>(x, dy, smem, smem + TK * dys, g, pl, it_begin, k0, c0, dys, win_h, win_w);
        if (ASYNC) cp_async_commit();
    }
    int stage = 0;
    for (int it = it_begin; it < it_end; ++it, stage ^= 1) {
        float* cur = smem + stage * stage_floats;
        if (it + 1 < it_end) {
            float* nxt = smem + (stage ^ 1) * stage_floats;
            stage_item<T, ASYNC, TK, TC>(x, dy, nxt, nxt + TK * dys, g, pl, it + 1, k0, c0, dys, win_h, win_w);
            if (ASYNC) { cp_async_commit(); cp_async_wait<1>(); }
        } else if (ASYNC) {
            cp_async_wait<0>();
        }
        __syncthreads();
        const float* s_dy = cur + otk * TKT * dys;
        const float* s_x = cur + TK * dys + otc * TCT;
        int pp = pg / pl.bq, qq = pg % pl.bq;
        for (int j = pg; j < npx; j += PG) {
            float d[TKT];
#pragma unroll
            for (int a = 0; a < TKT; ++a) d[a] = s_dy[a * dys + j];
            const float* xb = s_x + ((pp * g.stride_h) * win_w + qq * g.stride_w) * TC;
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int s = 0; s < S; ++s) {
                    Vec<TCT> xv;
                    xv.load(xb + (r * win_w + s) * TC);
#pragma unroll
                    for (int a = 0; a < TKT; ++a)
#pragma unroll
                        for (int b = 0; b < TCT; ++b)
                            acc[((a * TCT + b) * R + r) * S + s] = fmaf(d[a], xv.v[b], acc[((a * TCT + b) * R + r) * S + s]);
                }
            qq += PG;
            while (qq >= pl.bq) { qq -= pl.bq; ++pp; }
        }
        __syncthreads();    // everyone is done with this stage before it is refilled
    }

    // ---- sum the pixel groups: lanes first (groups that share a warp), then warps through shared memory ----
    constexpr int kWarps = kThreads / 32;
#pragma unroll
    for (int off = OT; off < 32; off <<= 1)
#pragma unroll
        for (int i = 0; i < ACC; ++i) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], off);
    // what is left per output thread: one partial sum per warp (OT < 32) or per pixel group (OT >= 32)
    constexpr int SETS = OT >= 32 ? PG : kWarps;
    constexpr int CH = 16;                                           // accumulators exchanged per pass
    __syncthreads();
    float* s_red = smem;                                             // [SETS][OT][CH]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool owner = OT >= 32 ? true : lane < OT;
    const int set = OT >= 32 ? pg : warp;
    float* out = pl.splits == 1 ? dw : partial + (size_t)split * g.k * g.c * R * S;
    const float scale = pl.splits == 1 ? g.alpha : 1.0f;
#pragma unroll
    for (int base = 0; base < ACC; base += CH) {
        if (owner) {
#pragma unroll
            for (int i = 0; i < CH; ++i)
                if (base + i < ACC) s_red[(set * OT + ot) * CH + i] = acc[base + i];
        }
        __syncthreads();
        for (int e = threadIdx.x; e < OT * CH; e += kThreads) {
            const int o = e / CH, i = e % CH, ai = base + i;
            if (ai < ACC) {
                float tot = 0.f;
#pragma unroll
                for (int w = 0; w < SETS; ++w) tot += s_red[(w * OT + o) * CH + i];
                const int a = ai / (TCT * R * S), b = (ai / (R * S)) % TCT, r = (ai / S) % R, s = ai % S;
                const int k = k0 + (o / OTC) * TKT + a, c = c0 + (o % OTC) * TCT + b;
                if (k < g.k && c < g.c) out[k * g.ws_k + c * g.ws_c + r * g.ws_r + s * g.ws_s] = scale * tot;
            }
        }
        __syncthreads();
    }
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

template <typename T> constexpr bool kAsyncOk = false;      // cp.async staging copies raw fp32
template <> constexpr bool kAsyncOk<float> = true;

// thread-tile shape of each variant
struct Variant { int tkt, tct, otk, otc; };
Variant variant_for(const Geom& g)
{
    const bool narrow = g.c <= 4;
    if (g.r == 5) return narrow ? Variant{1, 4, 16, 1} : Variant{2, 2, 8, 8};
    return narrow ? Variant{4, 4, 4, 1} : Variant{4, 4, 4, 4};
}

size_t smem_for(const Geom& g, const Variant& v, int bp, int bq)
{
    const int tk = v.tkt * v.otk, tc = v.tct * v.otc, ot = v.otk * v.otc;
    const size_t stage = 2 * sizeof(float) * ((size_t)tk * (bp * bq + 4) + (size_t)((bp - 1) * g.stride_h + g.r) * ((bq - 1) * g.stride_w + g.s) * tc);
    const int sets = ot >= 32 ? kThreads / ot : kThreads / 32;
    const size_t red = sizeof(float) * (size_t)sets * ot * 16;
    return stage > red ? stage : red;
}

template <typename T>
cudaError_t launch_t(const T* x, const T* dy, float* dw, float* partial, const Geom& g, const DirectPlan& pl,
                     cudaStream_t stream)
{
    if (!pl.tiled) {
        const long long total = (long long)g.k * g.r * g.s * g.c;
        direct_element_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(x, dy, dw, g);
        note_launch();
        return cudaGetLastError();
    }
    const Variant v = variant_for(g);
    const size_t smem = smem_for(g, v, pl.bp, pl.bq);
    dim3 grid(pl.tiles_k * pl.tiles_c, pl.splits);
    const bool use_async = kAsyncOk<T> && pl.vec_dy && pl.vec_x;
    bool done = false;
#define GACONV_DIRECT_CASE(RR, A, B, C, D)                                                                     \
    if (!done && g.r == RR && v.tkt == A && v.tct == B && v.otk == C && v.otc == D) {                          \
        if (use_async) {                                                                                       \
            if (smem > 48 * 1024) cudaFuncSetAttribute(direct_tiled_kernel<T, kAsyncOk<T>, RR, RR, A, B, C, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
            direct_tiled_kernel<T, kAsyncOk<T>, RR, RR, A, B, C, D><<<grid, kThreads, smem, stream>>>(x, dy, dw, partial, g, pl); \
        } else {                                                                                               \
            if (smem > 48 * 1024) cudaFuncSetAttribute(direct_tiled_kernel<T, false, RR, RR, A, B, C, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
            direct_tiled_kernel<T, false, RR, RR, A, B, C, D><<<grid, kThreads, smem, stream>>>(x, dy, dw, partial, g, pl); \
        }                                                                                                      \
        done = true;                                                                                           \
    }
    GACONV_DIRECT_CASE(1, 4, 4, 4, 4)
    GACONV_DIRECT_CASE(1, 4, 4, 4, 1)
    GACONV_DIRECT_CASE(3, 4, 4, 4, 4)
    GACONV_DIRECT_CASE(3, 4, 4, 4, 1)
    GACONV_DIRECT_CASE(5, 2, 2, 8, 8)
    GACONV_DIRECT_CASE(5, 1, 4, 16, 1)
#undef GACONV_DIRECT_CASE
    if (!done) return cudaErrorInvalidValue;
    note_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (pl.splits > 1) return reduce_splits(partial, dw, (size_t)g.k * g.c * g.r * g.s, pl.splits, g.alpha, stream);
    return cudaSuccess;
}

}  // namespace

DirectPlan plan_direct(const Geom& g)
{
    DirectPlan pl{};
    pl.tiled = (g.r == g.s) && (g.r == 1 || g.r == 3 || g.r == 5);
    const Variant v = variant_for(g);
    const int tk = v.tkt * v.otk, tc = v.tct * v.otc;
    pl.tiles_k = (g.k + tk - 1) / tk;
    pl.tiles_c = (g.c + tc - 1) / tc;
    pl.bq = g.q < 32 ? g.q : 32;
    pl.bp = 1;
    while (pl.bp * 2 <= g.p && pl.bp * 2 * pl.bq <= 128 && smem_for(g, v, pl.bp * 2, pl.bq) <= 64 * 1024) pl.bp *= 2;
    while (pl.bq > 1 && smem_for(g, v, pl.bp, pl.bq) > 64 * 1024) pl.bq /= 2;
    pl.bands_p = (g.p + pl.bp - 1) / pl.bp;
    pl.bands_q = (g.q + pl.bq - 1) / pl.bq;
    // vector fast paths: bands of whole rows whose pixel runs start on a 4-element boundary; NHWC with
    // channels a multiple of four (every 4-channel group is then aligned and entirely in or out of range)
    pl.vec_dy = pl.bq == g.q && g.p % pl.bp == 0 && (pl.bp * g.q) % 4 == 0;
    pl.vec_x = g.xs_c == 1 && g.c % 4 == 0 && tc % 4 == 0;
    pl.items = g.n * pl.bands_p * pl.bands_q;
    const int tiles = pl.tiles_k * pl.tiles_c;
    // one wave of two CTAs per SM (the register budget); each split's partial block is written once and read once
    int splits = (148 * 2) / tiles;
    if (splits < 1) splits = 1;
    if (splits > pl.items) splits = pl.items;
    const size_t out_bytes = (size_t)g.k * g.c * g.r * g.s * sizeof(float);
    while (splits > 1 && (size_t)splits * out_bytes > ((size_t)96 << 20)) --splits;
    if (splits < 1) splits = 1;
    {   // no empty splits
        const int per = (pl.items + splits - 1) / splits;
        splits = (pl.items + per - 1) / per;
    }
    if (!pl.tiled) splits = 1;
    pl.splits = splits;
    pl.partial_bytes = splits > 1 ? (size_t)splits * out_bytes : 0;
    return pl;
}

cudaError_t launch_direct(const void* x, const void* dy, float* dw, float* partial, uint32_t* counters,
                          const Geom& g, const DirectPlan& plan, cudaStream_t stream)
{
    (void)counters;
    if (g.bf16)
        return launch_t(static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(dy), dw, partial, g, plan, stream);
    return launch_t(static_cast<const float*>(x), static_cast<const float*>(dy), dw, partial, g, plan, stream);
}

}  // namespace gaconv
