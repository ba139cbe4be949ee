// Exact filter gradient on the FP32 pipes (paper Section 2.4: "to compute df we have to convolve I
// with dO"):   dW[k,c,r,s] = alpha * sum_{n,p,q} Xz[n,c,p*st+r-pad,q*st+s-pad] * dY[n,k,p,q].
// Works for every shape, layout and dtype: products and sums are fp32, so fp32 inputs meet the
// fp32 tolerance class.  It serves fp32 inputs, the 3-channel stem layers and every shape the
// tensor-core path does not tile.
//
// Register-tiled kernel.  A CTA owns a (TKT*OTK) x (TCT*OTC) block of (k, c) with all R*S filter
// taps, and a contiguous range of work items; an item is one image's band of BP x BQ output pixels.
// Per item the dY band ([k][pixel]) and the X window ([row][col][c]) are staged in shared memory
// as fp32, two stages deep: fp32 NHWC inputs arrive as TMA boxes (zero fill = padding) while the
// previous item is being consumed; other inputs are loaded and converted by the threads.  The OTK*OTC "output threads" of a pixel
// group each keep TKT*TCT*R*S accumulators in registers; the 128/(OTK*OTC) pixel groups take the
// band's pixels round-robin, so one vector load of dY and R*S vector loads of X feed
// TKT*TCT*R*S FMAs.  At the end the pixel groups are summed (warp shuffles, then shared memory, in a
// fixed order) and the CTA writes its block: to dW if it is the only split, else to its slot of
// the partial buffer, which reduce_splits() adds up in split order.
#include "gaconv_internal.h"
#include "device_utils.cuh"
#include "tma.cuh"

namespace gaconv {
namespace {

constexpr int kThreads = 128;

template <int N> struct Vec;
template <> struct Vec<1> { float v[1]; __device__ void load(const float* p) { v[0] = *p; } };
template <> struct Vec<2> { float v[2]; __device__ void load(const float* p) { float2 t = *reinterpret_cast<const float2*>(p); v[0] = t.x; v[1] = t.y; } };
template <> struct Vec<4> { float v[4]; __device__ void load(const float* p) { float4 t = *reinterpret_cast<const float4*>(p); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; } };

// Stage one work item with the CTA's threads: dY band as [k][pixel] (row stride dys) and X window as
// [row][col][TC], converted to fp32; four elements per load where the layout allows.
template <typename T, bool UNUSED, int TK, int TC>
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
            float v[4] = {0.f, 0.f, 0.f, 0.f};
            if (k < g.k) ld4(src, v);
            *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
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
                float v[4] = {0.f, 0.f, 0.f, 0.f};
                if (ok) ld4(xrow + (long long)ww * g.xs_w + c, v);
                *reinterpret_cast<float4*>(drow + i * 4) = make_float4(v[0], v[1], v[2], v[3]);
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

// STAGING: 0 = loads by the threads with conversion (any dtype/layout); 1 = TMA tiles (fp32, NHWC,
// C and P*Q multiples of four): one thread issues a 3-D box of dY and a 4-D box of X per item (zero
// fill outside the tensor gives the padding) and an mbarrier per stage signals arrival.
template <typename T, int STAGING, int R, int S, int TKT, int TCT, int OTK, int OTC>
__global__ void __launch_bounds__(kThreads)
direct_tiled_kernel(const T* __restrict__ x, const T* __restrict__ dy, float* __restrict__ dw,
                    float* __restrict__ partial, uint32_t* __restrict__ status,
                    const __grid_constant__ CUtensorMap map_dy, const __grid_constant__ CUtensorMap map_x,
                    Geom g, DirectPlan pl)
{
    constexpr int TK = TKT * OTK, TC = TCT * OTC, OT = OTK * OTC, PG = kThreads / OT, ACC = TKT * TCT * R * S;
    static_assert(kThreads % OT == 0 && OT <= 64, "output threads must divide the CTA");
    extern __shared__ __align__(128) float smem[];
    __shared__ __align__(8) uint64_t bar_full[2];
    __shared__ volatile int s_fail;
    const int npx = pl.bp * pl.bq;
    const int dys = STAGING == 1 ? npx : npx + 4;   // row stride of the dY band (TMA writes dense rows)
    const int win_h = (pl.bp - 1) * g.stride_h + R, win_w = (pl.bq - 1) * g.stride_w + S;
    const int stage_floats = (TK * dys + win_h * win_w * TC + 31) & ~31;   // stages start 128-byte aligned

    const int tile = blockIdx.x, split = blockIdx.y;
    const int k0 = (tile / pl.tiles_c) * TK, c0 = (tile % pl.tiles_c) * TC;
    const int ot = threadIdx.x % OT, pg = threadIdx.x / OT;
    const int otk = ot / OTC, otc = ot % OTC;

    float acc[ACC];
#pragma unroll
    for (int i = 0; i < ACC; ++i) acc[i] = 0.f;

    const int per = (pl.items + pl.splits - 1) / pl.splits;
    const int it_begin = split * per, it_end = min(pl.items, (split + 1) * per);
    const uint32_t tx_bytes = (uint32_t)(TK * npx + win_h * win_w * TC) * 4u;
    auto tma_issue = [&](int it, int stage) {     // one thread: both boxes of item `it` into `stage`
        const int n = it / (pl.bands_p * pl.bands_q);
        const int band = it % (pl.bands_p * pl.bands_q);
        const int p0 = (band / pl.bands_q) * pl.bp;
        const uint32_t full = smem_u32(&bar_full[stage]);
        const uint32_t dst = smem_u32(smem + stage * stage_floats);
        mbar_expect_tx(full, tx_bytes);
        tma_load_3d(dst, &map_dy, full, p0 * g.q, k0, n);
        tma_load_4d(dst + TK * npx * 4, &map_x, full, c0, -g.pad_w, p0 * g.stride_h - g.pad_h, n);
    };
    if (STAGING != 1) pdl_wait_prior_grid();
    if (STAGING == 1) {
        if (threadIdx.x == 0) {
            s_fail = 0;
            mbar_init(smem_u32(&bar_full[0]), 1); mbar_init(smem_u32(&bar_full[1]), 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncthreads();
        pdl_wait_prior_grid();
        if (threadIdx.x == 0 && it_begin < it_end) tma_issue(it_begin, 0);
    } else if (it_begin < it_end) {
        stage_item<T, false, TK, TC>(x, dy, smem, smem + TK * dys, g, pl, it_begin, k0, c0, dys, win_h, win_w);
    }
    int stage = 0;
    uint32_t phase[2] = {0u, 0u};
    for (int it = it_begin; it < it_end; ++it, stage ^= 1) {
        float* cur = smem + stage * stage_floats;
        if (it + 1 < it_end) {
            if (STAGING == 1) { if (threadIdx.x == 0) tma_issue(it + 1, stage ^ 1); }
            else {
                float* nxt = smem + (stage ^ 1) * stage_floats;
                stage_item<T, false, TK, TC>(x, dy, nxt, nxt + TK * dys, g, pl, it + 1, k0, c0, dys, win_h, win_w);
            }
        }
        if (STAGING == 1) {
            if (!mbar_wait(smem_u32(&bar_full[stage]), phase[stage])) s_fail = 1;   // bounded wait gave up
            phase[stage] ^= 1u;
            __syncthreads();
            if (s_fail) {                                                            // uniform exit
                if (threadIdx.x == 0) {
                    atomicOr(status, 1u);
                    // the next item's copies are already in flight: let them land (bounded) before the CTA's memory is released
                    if (it + 1 < it_end) (void)mbar_wait(smem_u32(&bar_full[stage ^ 1]), phase[stage ^ 1]);
                }
                __syncthreads();
                break;
            }
        } else {
            __syncthreads();
        }
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
    pdl_release_next_grid();
    pdl_wait_prior_grid();
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

template <typename T> constexpr bool kTmaOk = false;      // TMA staging copies raw fp32
template <> constexpr bool kTmaOk<float> = true;

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
    const size_t stage = 2 * sizeof(float) * ((((size_t)tk * (bp * bq + 4) + (size_t)((bp - 1) * g.stride_h + g.r) * ((bq - 1) * g.stride_w + g.s) * tc) + 31) & ~(size_t)31);
    const int sets = ot >= 32 ? kThreads / ot : kThreads / 32;
    const size_t red = sizeof(float) * (size_t)sets * ot * 16;
    return stage > red ? stage : red;
}

template <typename T>
cudaError_t launch_t(const T* x, const T* dy, float* dw, float* partial, uint32_t* status, const Geom& g,
                     const DirectPlan& pl, cudaStream_t stream)
{
    if (!pl.tiled) {
        const long long total = (long long)g.k * g.r * g.s * g.c;
        direct_element_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(x, dy, dw, g);
        note_launch();
        return cudaGetLastError();
    }
    const Variant v = variant_for(g);
    const int tk = v.tkt * v.otk, tc = v.tct * v.otc;
    const size_t smem = smem_for(g, v, pl.bp, pl.bq);
    dim3 grid(pl.tiles_k * pl.tiles_c, pl.splits);
    const int npx = pl.bp * pl.bq, pq = g.p * g.q;
    const int win_h = (pl.bp - 1) * g.stride_h + g.r, win_w = (pl.bq - 1) * g.stride_w + g.s;
    // TMA staging: fp32 tiles copied as they are
    bool use_tma = kTmaOk<T> && pl.vec_dy && pl.vec_x && pq % 4 == 0 && npx <= 256 && win_w <= 256 && win_h <= 256 &&
                   encode_fn() != nullptr;
    CUtensorMap map_dy{}, map_x{};
    if (use_tma) {
        cuuint64_t d3[3] = {(cuuint64_t)pq, (cuuint64_t)g.k, (cuuint64_t)g.n};
        cuuint64_t s3[2] = {(cuuint64_t)pq * 4, (cuuint64_t)g.k * pq * 4};
        cuuint32_t b3[3] = {(cuuint32_t)npx, (cuuint32_t)tk, 1}, e3[3] = {1, 1, 1};
        cuuint64_t d4[4] = {(cuuint64_t)g.c, (cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)g.n};
        cuuint64_t s4[3] = {(cuuint64_t)g.c * 4, (cuuint64_t)g.w * g.c * 4, (cuuint64_t)g.h * g.w * g.c * 4};
        cuuint32_t b4[4] = {(cuuint32_t)tc, (cuuint32_t)win_w, (cuuint32_t)win_h, 1}, e4[4] = {1, 1, 1, 1};
        if (encode_fn()(&map_dy, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<T*>(dy), d3, s3, b3, e3, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
            encode_fn()(&map_x, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<T*>(x), d4, s4, b4, e4, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            use_tma = false;
    }
    bool done = false;
    cudaError_t launch_err = cudaSuccess;
#define GACONV_DIRECT_LAUNCH(ST, RR, A, B, C, D)                                                                                 \
    {                                                                                                                            \
        auto kern = direct_tiled_kernel<T, ST, RR, RR, A, B, C, D>;                                                              \
        if (smem > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);                \
        launch_err = launch_kernel(kern, grid, dim3(kThreads), smem, stream, dim3(1, 1, 1), x, dy, dw, partial, status, map_dy, map_x, g, pl); \
    }
#define GACONV_DIRECT_CASE(RR, A, B, C, D)                                                                     \
    if (!done && g.r == RR && v.tkt == A && v.tct == B && v.otk == C && v.otc == D) {                          \
        if (use_tma) GACONV_DIRECT_LAUNCH(kTmaOk<T> ? 1 : 0, RR, A, B, C, D)                                   \
        else GACONV_DIRECT_LAUNCH(0, RR, A, B, C, D)                                                           \
        done = true;                                                                                           \
    }
    GACONV_DIRECT_CASE(1, 4, 4, 4, 4)
    GACONV_DIRECT_CASE(1, 4, 4, 4, 1)
    GACONV_DIRECT_CASE(3, 4, 4, 4, 4)
    GACONV_DIRECT_CASE(3, 4, 4, 4, 1)
    GACONV_DIRECT_CASE(5, 2, 2, 8, 8)
    GACONV_DIRECT_CASE(5, 1, 4, 16, 1)
#undef GACONV_DIRECT_CASE
#undef GACONV_DIRECT_LAUNCH
    if (!done) return cudaErrorInvalidValue;
    note_launch();
    if (launch_err != cudaSuccess) return launch_err;
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
    // few input channels: the items are cheap and staged by the threads themselves, so a CTA takes its whole
    // share as one or two large items (one exposed load latency instead of four)
    const int max_px = g.c <= 4 ? 512 : 128;
    while (pl.bp * 2 <= g.p && pl.bp * 2 * pl.bq <= max_px && smem_for(g, v, pl.bp * 2, pl.bq) <= 96 * 1024) pl.bp *= 2;
    while (pl.bq > 1 && smem_for(g, v, pl.bp, pl.bq) > 96 * 1024) pl.bq /= 2;
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

cudaError_t launch_direct(const void* x, const void* dy, float* dw, float* partial, uint32_t* status,
                          const Geom& g, const DirectPlan& plan, cudaStream_t stream)
{
    if (g.bf16)
        return launch_t(static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(dy), dw, partial, status, g, plan, stream);
    return launch_t(static_cast<const float*>(x), static_cast<const float*>(dy), dw, partial, status, g, plan, stream);
}

}  // namespace gaconv
