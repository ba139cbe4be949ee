// Exact filter gradient of fp32 inputs on the warp-level tensor-core path: mma.sync m16n8k8,
// TF32 operands, fp32 accumulate, with the operands split so that fp32 accuracy is kept:
//   x = big + small,  big = tf32(x) (by truncation),  small = tf32(x - big)
//   a*b ~= big_a*big_b + big_a*small_b + small_a*big_b            ("3xTF32": error ~ 2^-21 per product)
// One pass (big*big only) is the opt-in GACONV_MATH_TF32 mode: operands cut to 10 mantissa bits.
// (bf16 inputs take the tcgen05 kernel, which measured faster wherever both tile the shape, or the FP32 pipes.)
//
//   dW[k,c,r,s] = alpha * sum_{n,p,q} Xz[n,c,p*st+r-pad,q*st+s-pad] * dY[n,k,p,q]              (Section 2.4)
//
// Same decomposition as the FP32-pipe kernel: a CTA owns a 16 (k) x 16 (c) block with all R*S taps and a
// range of work items (an item = one image's band of whole output rows); the dY band and the X window
// arrive as fp32 TMA boxes in two shared-memory stages.  Per 8 pixels (one MMA k-step) a warp loads the
// 16x8 dY fragment once and, for each tap and each half of the 16 channels, an 8x8 X fragment, splits
// both in registers and issues three MMAs into the tap's accumulator.  For 1x1 and 3x3 filters the four
// warps of a CTA take the k-steps round-robin and their accumulators are added through shared memory in
// warp order; for 5x5 they split the 25 taps instead (register budget).  Splits: reduce_splits().
//   dY box: 32 pixels x 16 channels with the 128-byte TMA swizzle, so that the eight k-rows a fragment
//   load touches fall in different banks.
#include "gaconv_internal.h"
#include "device_utils.cuh"
#include "tma.cuh"

namespace gaconv {
namespace {

constexpr int kThreads = 128, kWarps = 4, TK = 16, TC = 16;

template <int R, int S, bool THREE_PASS>
__global__ void __launch_bounds__(kThreads)
direct_mma_kernel(float* __restrict__ dw, float* __restrict__ partial, uint32_t* __restrict__ status,
                  const __grid_constant__ CUtensorMap map_dy, const __grid_constant__ CUtensorMap map_x,
                  Geom g, DirectPlan pl)
{
    constexpr int TAPS = R * S;
    // Up to 9 taps: every warp holds all taps and the warps split the k-steps (their accumulators are added at
    // the end).  More taps (5x5): the accumulators would not fit the register file, so the warps split the
    // TAPS instead -- each runs all k-steps for its own taps, and no cross-warp sum is needed.
    constexpr bool SPLIT_TAPS = TAPS > 9;
    constexpr int TPW = SPLIT_TAPS ? (TAPS + kWarps - 1) / kWarps : TAPS;   // taps per warp
    constexpr int NT = TPW * 2;                          // n-tiles of 8 channels: tap-major, channel half minor
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[2];
    __shared__ volatile int s_fail;

    const int npx = pl.bp * pl.bq;                       // a multiple of 32; bq == Q, a multiple of 8
    const int win_h = (pl.bp - 1) * g.stride_h + R, win_w = (pl.bq - 1) * g.stride_w + S;
    constexpr int EB = 4, BOXPX = 32, KPX = 8;
    const int dy_bytes = npx / BOXPX * 2048;             // [boxes][16 k][128-byte swizzled rows]
    const int x_bytes = win_h * win_w * TC * EB;         // [row][col][16 c]
    const int stage_bytes = (dy_bytes + x_bytes + 1023) & ~1023;
    uint8_t* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);

    const int tile = blockIdx.x, split = blockIdx.y;
    const int k0 = (tile / pl.tiles_c) * TK, c0 = (tile % pl.tiles_c) * TC;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gq = lane >> 2, tq = lane & 3;

    float acc[NT][4];
#pragma unroll
    for (int i = 0; i < NT; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
    const int tap_lo = SPLIT_TAPS ? warp * TPW : 0;      // first tap of this warp

    const int per = (pl.items + pl.splits - 1) / pl.splits;
    const int it_begin = split * per, it_end = min(pl.items, (split + 1) * per);
    auto tma_issue = [&](int it, int stage) {
        const int n = it / pl.bands_p, p0 = (it % pl.bands_p) * pl.bp;
        const uint32_t full = smem_u32(&bar_full[stage]);
        const uint32_t dst = smem_u32(smem + stage * stage_bytes);
        mbar_expect_tx(full, (uint32_t)(dy_bytes + x_bytes));
        for (int b = 0; b < npx / BOXPX; ++b) tma_load_3d(dst + b * 2048, &map_dy, full, p0 * g.q + BOXPX * b, k0, n);
        tma_load_4d(dst + dy_bytes, &map_x, full, c0, -g.pad_w, p0 * g.stride_h - g.pad_h, n);
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
        const float* s_x = reinterpret_cast<const float*>(s_dy + dy_bytes);

        for (int ks = SPLIT_TAPS ? 0 : warp; ks < npx / KPX; ks += SPLIT_TAPS ? 1 : kWarps) {
            const int px0 = ks * KPX;
            // ---- A fragment: dY[k = gq (+8)][px0 + tq (+4)], from the swizzled box ----
            uint32_t a_big[4], a_small[4];
            {
                const uint8_t* box = s_dy + (px0 >> 5) * 2048;
                const int ch0 = (px0 & 31) >> 2;                 // 16-byte chunk of px0 within its 128-byte row
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int row = gq + (i & 1) * 8, ch = ch0 + (i >> 1);
                    const float v = *reinterpret_cast<const float*>(box + row * 128 + ((ch ^ (row & 7)) << 4) + tq * 4);
                    a_big[i] = to_tf32(v);
                    if (THREE_PASS) a_small[i] = to_tf32(v - __uint_as_float(a_big[i]));
                }
            }
            // ---- B fragments: X[pixel px0 + tq (+4) shifted by the tap][c = half*8 + gq] ----
            const int pp = px0 / pl.bq, qq = px0 - pp * pl.bq;   // the 8 pixels share an output row
            const float* xrow = s_x + ((pp * g.stride_h) * win_w + (qq + tq) * g.stride_w) * TC + gq;
            const int px4 = 4 * g.stride_w * TC;                 // four pixels further along the row
#pragma unroll
            for (int i = 0; i < TPW; ++i) {
                const int tap = tap_lo + i;
                if (SPLIT_TAPS && tap >= TAPS) break;
                const int r = SPLIT_TAPS ? tap / S : i / S, s = SPLIT_TAPS ? tap % S : i % S;
                const float* xt = xrow + (r * win_w + s) * TC;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const float v0 = xt[h * 8], v1 = xt[h * 8 + px4];
                    const uint32_t b0 = to_tf32(v0), b1 = to_tf32(v1);
                    float (&d)[4] = acc[i * 2 + h];
                    if (THREE_PASS) {
                        const uint32_t s0 = to_tf32(v0 - __uint_as_float(b0)), s1 = to_tf32(v1 - __uint_as_float(b1));
                        mma_tf32(d, a_small, b0, b1);
                        mma_tf32(d, a_big, s0, s1);
                    }
                    mma_tf32(d, a_big, b0, b1);
                }
            }
        }
        __syncthreads();    // everyone is done with this stage before it is refilled
    }

    // ---- add the four warps' accumulators in warp order, then write the block ----
    // s_red[warp][k][tap][c]: thread (gq, tq) holds rows gq, gq+8 and columns 2*tq, 2*tq+1 of each n-tile
    float* s_red = reinterpret_cast<float*>(smem);
    constexpr int BLK = TK * TAPS * TC;
    constexpr int SLOTS = SPLIT_TAPS ? 1 : kWarps;       // split taps: the warps own disjoint columns of one block
#pragma unroll
    for (int i = 0; i < NT; ++i) {
        const int tap = tap_lo + (i >> 1), cbase = (i & 1) * 8 + 2 * tq;
        if (SPLIT_TAPS && tap >= TAPS) continue;
        float* base = s_red + (SPLIT_TAPS ? 0 : warp * BLK);
        *reinterpret_cast<float2*>(base + (gq * TAPS + tap) * TC + cbase) = make_float2(acc[i][0], acc[i][1]);
        *reinterpret_cast<float2*>(base + ((gq + 8) * TAPS + tap) * TC + cbase) = make_float2(acc[i][2], acc[i][3]);
    }
    __syncthreads();
    float* out = pl.splits == 1 ? dw : partial + (size_t)split * g.k * g.c * R * S;
    const float scale = pl.splits == 1 ? g.alpha : 1.0f;
    for (int e = threadIdx.x; e < BLK; e += kThreads) {
        float tot = s_red[e];
#pragma unroll
        for (int w = 1; w < SLOTS; ++w) tot += s_red[w * BLK + e];
        const int cc = e % TC, tap = (e / TC) % TAPS, kk = e / (TC * TAPS);
        const int k = k0 + kk, c = c0 + cc;
        if (k < g.k && c < g.c) out[k * g.ws_k + c * g.ws_c + (tap / S) * g.ws_r + (tap % S) * g.ws_s] = scale * tot;
    }
}

}  // namespace

bool direct_mma_supported(const Geom& g, const DirectPlan& pl)
{
    if (g.bf16 || g.xs_c != 1 || g.c % 4 != 0 || g.c < 8) return false;
    if (g.r != g.s || (g.r != 1 && g.r != 3 && g.r != 5)) return false;
    const int npx = pl.bp * pl.bq, pq = g.p * g.q;
    const int boxpx = 32, kpx = 8;
    if (pl.bq != g.q || g.q % kpx != 0 || g.p % pl.bp != 0 || npx % boxpx != 0 || npx > 256 || pq % 8 != 0) return false;
    const int win_h = (pl.bp - 1) * g.stride_h + g.r, win_w = (pl.bq - 1) * g.stride_w + g.s;
    if (win_h > 256 || win_w > 256) return false;
    return encode_fn() != nullptr;
}

cudaError_t launch_direct_mma(const void* x, const void* dy, float* dw, float* partial, uint32_t* status, const Geom& g,
                              const DirectPlan& pl, bool three_pass, cudaStream_t stream)
{
    const int npx = pl.bp * pl.bq, pq = g.p * g.q;
    const int win_h = (pl.bp - 1) * g.stride_h + g.r, win_w = (pl.bq - 1) * g.stride_w + g.s;
    CUtensorMap map_dy, map_x;
    cuuint64_t d3[3] = {(cuuint64_t)pq, (cuuint64_t)g.k, (cuuint64_t)g.n};
    const int eb = 4, boxpx = 32;
    const CUtensorMapDataType dt = CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    cuuint64_t s3[2] = {(cuuint64_t)pq * eb, (cuuint64_t)g.k * pq * eb};
    cuuint32_t b3[3] = {(cuuint32_t)boxpx, (cuuint32_t)TK, 1}, e3[3] = {1, 1, 1};
    cuuint64_t d4[4] = {(cuuint64_t)g.c, (cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)g.n};
    cuuint64_t s4[3] = {(cuuint64_t)g.c * eb, (cuuint64_t)g.w * g.c * eb, (cuuint64_t)g.h * g.w * g.c * eb};
    cuuint32_t b4[4] = {(cuuint32_t)TC, (cuuint32_t)win_w, (cuuint32_t)win_h, 1}, e4[4] = {1, 1, 1, 1};
    if (encode_fn()(&map_dy, dt, 3, const_cast<void*>(dy), d3, s3, b3, e3, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
        encode_fn()(&map_x, dt, 4, const_cast<void*>(x), d4, s4, b4, e4, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    const size_t stage = ((size_t)(npx / boxpx) * 2048 + (size_t)win_h * win_w * TC * eb + 1023) & ~(size_t)1023;
    const size_t red = (size_t)(g.r * g.s > 9 ? 1 : kWarps) * TK * g.r * g.s * TC * 4;
    size_t smem = 2 * stage > red ? 2 * stage : red;
    smem += 1024;
    dim3 grid(pl.tiles_k * pl.tiles_c, pl.splits);
    cudaError_t launch_err = cudaErrorInvalidValue;
#define GACONV_MMA_CASE(RR, TP)                                                                                          \
    if (g.r == RR && three_pass == TP) {                                                                                 \
        auto kern = direct_mma_kernel<RR, RR, TP>;                                                                       \
        if (smem > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);        \
        launch_err = launch_kernel(kern, grid, dim3(kThreads), smem, stream, dim3(1, 1, 1), dw, partial, status, map_dy, map_x, g, pl); \
    }
    GACONV_MMA_CASE(1, true)
    GACONV_MMA_CASE(1, false)
    GACONV_MMA_CASE(3, true)
    GACONV_MMA_CASE(3, false)
    GACONV_MMA_CASE(5, true)
    GACONV_MMA_CASE(5, false)
#undef GACONV_MMA_CASE
    note_launch();
    if (launch_err != cudaSuccess) return launch_err;
    if (pl.splits > 1) return reduce_splits(partial, dw, (size_t)g.k * g.c * g.r * g.s, pl.splits, g.alpha, stream);
    return cudaSuccess;
}

}  // namespace gaconv
