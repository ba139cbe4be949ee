// Exact filter gradient for layers with very few input channels (the 3-channel stem convolutions) on the
// warp-level tensor-core path.
//
//   dW[k,c,r,s] = alpha * sum_{n,p,q} Xz[n,c,p*st+r-pad,q*st+s-pad] * dY[n,k,p,q]              (Section 2.4)
//
// With C = 3 neither operand format of the big kernels applies (a pixel is 6 or 12 bytes: no TMA box over
// channels, no 16-byte vectors).  But in NHWC the S*C values a filter row needs for output pixel q are
// CONTIGUOUS in the image row: X[n, h, (q*st - pad)*C .. + S*C).  So the image row is treated as a flat
// vector of W*C elements (its byte stride IS a multiple of 16), TMA-loaded with zero fill left and right
// (= padding), and the GEMM is  D[k, j] = sum_px dY[k, px] * B[px, j],  j = (r, s, c) flattened (R*S*C
// columns, padded to a multiple of 8), with  B[px, j] = Xrow[p*st + r][(q*st - pad)*C + s*C + c].
// A CTA owns 16 output channels, all columns and a range of work items (image bands of whole rows); its
// four warps take the 8- or 16-pixel k-steps round-robin.
//   fp32 inputs: mma.sync m16n8k8 TF32 on split operands (big + small, three MMAs: fp32 accuracy).
//   bf16 inputs: mma.sync m16n8k16 bf16 (products exact in fp32).
// Split partial blocks are added by reduce_splits() in split order.
#include <cstring>

#include "gaconv_internal.h"
#include "device_utils.cuh"
#include "tma.cuh"

namespace gaconv {
namespace {

constexpr int kThreads = 128, kWarps = 4, TK = 16;
constexpr int kMaxNT = 10;                                  // up to 80 flattened columns (5x5x3 = 75)

struct StemParams {
    Geom g;
    int tiles_k, bp, bands_p, items, splits;
    int box_px;        // pixels per dY box: 32 (fp32) or 64 (bf16), one 128-byte row per channel
    int box_w;         // elements per staged X row
    int x_start;       // flat coordinate of its first element (negative: left padding, aligned to 16 bytes)
    int lead;          // elements between the row start and flat position -pad*C
    int win_h, nt;     // staged rows per item; n-tiles of 8 columns
};


template <typename T, int NT>
__global__ void __launch_bounds__(kThreads)
stem_mma_kernel(float* __restrict__ dw, float* __restrict__ partial, uint32_t* __restrict__ status,
                const __grid_constant__ CUtensorMap map_dy, const __grid_constant__ CUtensorMap map_x, const StemParams P)
{
    constexpr bool F32 = sizeof(T) == 4;
    constexpr int KPX = F32 ? 8 : 16;                      // pixels per MMA k-step
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[2];
    __shared__ volatile int s_fail;
    const Geom& g = P.g;

    const int npx = P.bp * g.q;
    const int dy_bytes = npx / P.box_px * 2048;            // [boxes][16 k][128-byte swizzled rows]
    const int x_bytes = P.win_h * P.box_w * (int)sizeof(T);
    const int stage_bytes = (dy_bytes + x_bytes + 1023) & ~1023;
    uint8_t* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);

    const int k0 = blockIdx.x * TK, split = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gq = lane >> 2, tq = lane & 3;
    const int ncols = g.r * g.s * g.c, sc_per_row = g.s * g.c;

    // this thread's B columns: j = 8*h + gq  ->  offset of (r, s*C + c) inside the staged window, or -1
    int col_off[NT];
#pragma unroll
    for (int h = 0; h < NT; ++h) {
        const int j = 8 * h + gq;
        col_off[h] = j < ncols ? (j / sc_per_row) * P.box_w + (j % sc_per_row) + P.lead : -1;
    }
    float acc[NT][4];
#pragma unroll
    for (int i = 0; i < NT; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;

    const int per = (P.items + P.splits - 1) / P.splits;
    const int it_begin = split * per, it_end = min(P.items, (split + 1) * per);
    auto tma_issue = [&](int it, int stage) {
        const int n = it / P.bands_p, p0 = (it % P.bands_p) * P.bp;
        const uint32_t full = smem_u32(&bar_full[stage]);
        const uint32_t dst = smem_u32(smem + stage * stage_bytes);
        mbar_expect_tx(full, (uint32_t)(dy_bytes + x_bytes));
        for (int b = 0; b < npx / P.box_px; ++b) tma_load_3d(dst + b * 2048, &map_dy, full, p0 * g.q + P.box_px * b, k0, n);
        tma_load_3d(dst + dy_bytes, &map_x, full, P.x_start, p0 * g.stride_h - g.pad_h, n);
    };
    if (threadIdx.x == 0) {
        s_fail = 0;
        mbar_init(smem_u32(&bar_full[0]), 1); mbar_init(smem_u32(&bar_full[1]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pdl_wait_prior_grid();
    if (threadIdx.x == 0 && it_begin < it_end) tma_issue(it_begin, 0);

    int stage = 0;
    uint32_t phase0 = 0, phase1 = 0;
    for (int it = it_begin; it < it_end; ++it, stage ^= 1) {
        if (it + 1 < it_end && threadIdx.x == 0) tma_issue(it + 1, stage ^ 1);
        const uint32_t ph = stage ? phase1 : phase0;
        if (!mbar_wait(smem_u32(&bar_full[stage]), ph)) s_fail = 1;          // bounded wait gave up
        if (stage) phase1 ^= 1u; else phase0 ^= 1u;
        __syncthreads();
        if (s_fail) {                                                        // uniform exit
            if (threadIdx.x == 0) {
                atomicOr(status, 1u);
                // the next item's copies are already in flight: let them land (bounded) before the CTA's memory is released
                if (it + 1 < it_end) (void)mbar_wait(smem_u32(&bar_full[stage ^ 1]), stage ? phase0 : phase1);
            }
            __syncthreads();
            break;
        }
        const uint8_t* s_dy = smem + stage * stage_bytes;
        const T* s_x = reinterpret_cast<const T*>(s_dy + dy_bytes);

        for (int ks = warp; ks < npx / KPX; ks += kWarps) {
            const int px0 = ks * KPX;
            const int pp = px0 / g.q, qq = px0 - pp * g.q;                    // the k-step's pixels share an output row
            const uint8_t* box = s_dy + (px0 / P.box_px) * 2048;
            const int in_box = px0 % P.box_px;
            if constexpr (F32) {
                // A: dY[k = gq (+8)][px0 + tq (+4)]
                uint32_t a_big[4], a_small[4];
                const int ch0 = in_box >> 2;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = gq + (i & 1) * 8, ch = ch0 + (i >> 1);
                    const float v = *reinterpret_cast<const float*>(box + row * 128 + ((ch ^ (row & 7)) << 4) + tq * 4);
                    a_big[i] = to_tf32(v);
                    a_small[i] = to_tf32(v - __uint_as_float(a_big[i]));
                }
                // B: rows px0 + tq and px0 + tq + 4
                const float* x0 = reinterpret_cast<const float*>(s_x) + (pp * g.stride_h) * P.box_w + ((qq + tq) * g.stride_w) * g.c;
                const int px4 = 4 * g.stride_w * g.c;
#pragma unroll
                for (int h = 0; h < NT; ++h) {
                    const int o = col_off[h];
                    const float v0 = o >= 0 ? x0[o] : 0.f, v1 = o >= 0 ? x0[o + px4] : 0.f;
                    const uint32_t b0 = to_tf32(v0), b1 = to_tf32(v1);
                    const uint32_t s0 = to_tf32(v0 - __uint_as_float(b0)), s1 = to_tf32(v1 - __uint_as_float(b1));
                    mma_tf32(acc[h], a_small, b0, b1);
                    mma_tf32(acc[h], a_big, s0, s1);
                    mma_tf32(acc[h], a_big, b0, b1);
                }
            } else {
                // A: dY[k = gq (+8)][px0 + 2*tq, +1 (+8, +9)], two bf16 per register
                uint32_t a[4];
                const int ch0 = in_box >> 3;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = gq + (i & 1) * 8, ch = ch0 + (i >> 1);
                    a[i] = *reinterpret_cast<const uint32_t*>(box + row * 128 + ((ch ^ (row & 7)) << 4) + tq * 4);
                }
                // B: {B[2tq][j], B[2tq+1][j]} and the same eight pixels further
                const unsigned short* x0 = reinterpret_cast<const unsigned short*>(s_x) + (pp * g.stride_h) * P.box_w +
                                           ((qq + 2 * tq) * g.stride_w) * g.c;
                const int px1 = g.stride_w * g.c, px8 = 8 * px1;
#pragma unroll
                for (int h = 0; h < NT; ++h) {
                    const int o = col_off[h];
                    uint32_t b0 = 0u, b1 = 0u;
                    if (o >= 0) {
                        b0 = (uint32_t)x0[o] | ((uint32_t)x0[o + px1] << 16);
                        b1 = (uint32_t)x0[o + px8] | ((uint32_t)x0[o + px8 + px1] << 16);
                    }
                    mma_bf16(acc[h], a, b0, b1);
                }
            }
        }
        __syncthreads();    // everyone is done with this stage before it is refilled
    }

    // ---- add the four warps' accumulators in warp order, then write the block ----
    float* s_red = reinterpret_cast<float*>(smem);            // [warp][16 k][NT*8 columns]
    constexpr int NCOL = NT * 8, BLK = TK * NCOL;
#pragma unroll
    for (int h = 0; h < NT; ++h) {
        float* w0 = s_red + warp * BLK + gq * NCOL + 8 * h + 2 * tq;
        float* w1 = s_red + warp * BLK + (gq + 8) * NCOL + 8 * h + 2 * tq;
        *reinterpret_cast<float2*>(w0) = make_float2(acc[h][0], acc[h][1]);
        *reinterpret_cast<float2*>(w1) = make_float2(acc[h][2], acc[h][3]);
    }
    __syncthreads();
    float* out = P.splits == 1 ? dw : partial + (size_t)split * g.k * ncols;
    const float scale = P.splits == 1 ? g.alpha : 1.0f;
    for (int e = threadIdx.x; e < BLK; e += kThreads) {
        const int kk = e / NCOL, j = e % NCOL, k = k0 + kk;
        if (j >= ncols || k >= g.k) continue;
        float tot = s_red[e];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) tot += s_red[w * BLK + e];
        const int r = j / sc_per_row, sc = j % sc_per_row, s = sc / g.c, c = sc % g.c;
        out[k * g.ws_k + c * g.ws_c + r * g.ws_r + s * g.ws_s] = scale * tot;
    }
}

bool make_params(const Geom& g, StemParams* out)
{
    if (g.xs_c != 1 || g.c > 4) return false;                                  // NHWC, a handful of channels
    const int eb = g.bf16 ? 2 : 4, al = 16 / eb;
    const int ncols = g.r * g.s * g.c;
    if (ncols > 8 * kMaxNT || g.stride_h != g.stride_w) return false;
    if (((size_t)g.w * g.c * eb) % 16 != 0 || ((size_t)g.p * g.q * eb) % 16 != 0) return false;
    StemParams P{};
    P.g = g;
    P.box_px = g.bf16 ? 64 : 32;
    const int kpx = g.bf16 ? 16 : 8;
    if (g.q % kpx != 0) return false;
    // band: whole rows, a multiple of box_px pixels, at most 256
    int bp = 1;
    while ((bp * g.q) % P.box_px != 0) ++bp;
    if (bp > g.p || g.p % bp != 0 || bp * g.q > 256) return false;
    while (bp * 2 * g.q <= 256 && g.p % (bp * 2) == 0) bp *= 2;
    P.bp = bp;
    P.bands_p = g.p / bp;
    P.items = g.n * P.bands_p;
    P.tiles_k = (g.k + TK - 1) / TK;
    const int flat0 = -g.pad_w * g.c;
    P.x_start = flat0 >= 0 ? flat0 / al * al : -((-flat0 + al - 1) / al * al);
    P.lead = flat0 - P.x_start;
    const int win_w = (g.q - 1) * g.stride_w + g.s;
    const int need = P.lead + win_w * g.c;
    P.box_w = (need + al - 1) / al * al;
    P.win_h = (bp - 1) * g.stride_h + g.r;
    if (P.box_w > 256 || P.win_h > 256) return false;
    P.nt = (ncols + 7) / 8;
    int splits = (148 * (ncols <= 32 ? 8 : 4)) / P.tiles_k;     // (3x3 stems: eight light CTAs per SM hide the fragment latency better)
    if (splits < 1) splits = 1;
    if (splits > P.items) splits = P.items;
    const int per = (P.items + splits - 1) / splits;
    P.splits = (P.items + per - 1) / per;
    *out = P;
    return true;
}

template <typename T>
cudaError_t launch_t(const void* x, const void* dy, float* dw, float* partial, uint32_t* status, const StemParams& P,
                     cudaStream_t stream)
{
    const Geom& g = P.g;
    const int eb = (int)sizeof(T), pq = g.p * g.q;
    const CUtensorMapDataType dt = eb == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    CUtensorMap map_dy, map_x;
    cuuint64_t d3[3] = {(cuuint64_t)pq, (cuuint64_t)g.k, (cuuint64_t)g.n};
    cuuint64_t s3[2] = {(cuuint64_t)pq * eb, (cuuint64_t)g.k * pq * eb};
    cuuint32_t b3[3] = {(cuuint32_t)P.box_px, (cuuint32_t)TK, 1}, e3[3] = {1, 1, 1};
    cuuint64_t dx[3] = {(cuuint64_t)g.w * g.c, (cuuint64_t)g.h, (cuuint64_t)g.n};
    cuuint64_t sx[2] = {(cuuint64_t)g.w * g.c * eb, (cuuint64_t)g.h * g.w * g.c * eb};
    cuuint32_t bx[3] = {(cuuint32_t)P.box_w, (cuuint32_t)P.win_h, 1};
    if (encode_fn()(&map_dy, dt, 3, const_cast<void*>(dy), d3, s3, b3, e3, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
        encode_fn()(&map_x, dt, 3, const_cast<void*>(x), dx, sx, bx, e3, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    const int npx = P.bp * g.q;
    const size_t stage = ((size_t)(npx / P.box_px) * 2048 + (size_t)P.win_h * P.box_w * eb + 1023) & ~(size_t)1023;
    const size_t red = (size_t)kWarps * TK * P.nt * 8 * 4;
    size_t smem = (2 * stage > red ? 2 * stage : red) + 1024;
    dim3 grid(P.tiles_k, P.splits);
    cudaError_t err = cudaErrorInvalidValue;
#define GACONV_STEM_CASE(N)                                                                                        \
    if (P.nt == N) {                                                                                               \
        auto kern = stem_mma_kernel<T, N>;                                                                         \
        if (smem > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  \
        err = launch_kernel(kern, grid, dim3(kThreads), smem, stream, dim3(1, 1, 1), dw, partial, status, map_dy, map_x, P); \
    }
    GACONV_STEM_CASE(1) GACONV_STEM_CASE(2) GACONV_STEM_CASE(3) GACONV_STEM_CASE(4) GACONV_STEM_CASE(5)
    GACONV_STEM_CASE(6) GACONV_STEM_CASE(7) GACONV_STEM_CASE(8) GACONV_STEM_CASE(9) GACONV_STEM_CASE(10)
#undef GACONV_STEM_CASE
    note_launch();
    if (err != cudaSuccess) return err;
    if (P.splits > 1) return reduce_splits(partial, dw, (size_t)g.k * g.c * g.r * g.s, P.splits, g.alpha, stream);
    return cudaSuccess;
}

}  // namespace

bool plan_stem(const Geom& g, StemPlan* plan)
{
    StemParams P;
    if (!make_params(g, &P) || encode_fn() == nullptr) return false;
    plan->partial_bytes = P.splits > 1 ? (size_t)P.splits * g.k * g.c * g.r * g.s * sizeof(float) : 0;
    static_assert(sizeof(StemParams) <= sizeof(plan->opaque), "StemPlan::opaque too small");
    memcpy(plan->opaque, &P, sizeof(P));
    return true;
}

cudaError_t launch_stem(const void* x, const void* dy, float* dw, float* partial, uint32_t* status, const StemPlan& plan,
                        cudaStream_t stream)
{
    StemParams P;
    memcpy(&P, plan.opaque, sizeof(P));
    return P.g.bf16 ? launch_t<__nv_bfloat16>(x, dy, dw, partial, status, P, stream)
                    : launch_t<float>(x, dy, dw, partial, status, P, stream);
}

}  // namespace gaconv
