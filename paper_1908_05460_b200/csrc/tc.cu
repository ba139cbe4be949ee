// Exact filter gradient as an implicit GEMM on the 5th-generation tensor cores (tcgen05), for sm_100a.
//
//   dW[k, r, s, c] = alpha * sum_{n,p,q} dY[n,k,p,q] * Xz[n, p*st+r-pad, q*st+s-pad, c]      (Section 2.4)
//
// GEMM view per filter row r:  D_r[k, (s,c)] = sum_j A[k, j] * B_r[(s,c), j],  j = (n,p,q).
//   A  = dY in its own layout [n][k][pq]: for a fixed image the k x pq block is K-major (the
//        reduction index is contiguous), loaded by TMA into 128-/64-/32-byte swizzled rows.
//   B  = X in NHWC: for a fixed shift (r,s) the pixel x channel block is MN-major (channels
//        contiguous).  One TMA tile per column shift s (zero fill outside the image gives the
//        padding for free); the S tiles sit at a uniform stride in shared memory, so a single MMA
//        of N = S*CT columns covers all column shifts (the stride is the descriptor's leading
//        byte offset).  For stride 1 the row shift r is a row offset into a tile that carries
//        R-1 halo rows ("halo" mode); otherwise every (r,s) has its own tile ("separate" mode).
//   D  = R accumulators in tensor memory, fp32.  With M = 64 (K <= 64) an accumulator occupies 16 of
//        the 32 lanes of each TMEM sub-partition, so two accumulators share the same columns.
// A CTA owns one (k-tile, c-tile) block of dW and a contiguous range of reduction chunks; the
// partial blocks of the splits are combined by the last CTA to finish, in split order.
//
// Warp roles: warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer, warps 2..5 = epilogue.
// Every mbarrier wait is bounded; on expiry the kernel raises the workspace status word, drains
// the copies it has in flight, frees its tensor memory and returns.
#include <cuda.h>

#include <cstdlib>
#include <cstring>

#include "gaconv_internal.h"

namespace gaconv {
namespace {

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit expires.
constexpr uint32_t kWaitLimit = 1u << 22;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitLimit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&v)[16]) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor: start address, leading/stride byte offsets (16-byte units),
// descriptor version 1, swizzle code in bits 61..63 (2 = 128 B, 4 = 64 B, 6 = 32 B).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo, uint32_t swz_code) {
    return (uint64_t)((addr >> 4) & 0x3fffu) | ((uint64_t)((lbo >> 4) & 0x3fffu) << 16) |
           ((uint64_t)((sbo >> 4) & 0x3fffu) << 32) | (1ull << 46) | ((uint64_t)swz_code << 61);
}

struct TcParams {
    Geom g;
    int m;              // MMA M: 64 or 128 output channels per k-tile
    int kb;             // rows of an A box (k rounded up to 8, at most m)
    int ct;             // input channels per c-tile; MMA N = s * ct
    int tiles_k, tiles_c, splits;
    int halo;           // 1: S tiles with R-1 halo rows, row shift = row offset; 0: R*S tiles
    int ci, bp;         // chunk = ci images x bp output rows (ci > 1 only when the map has < 64 pixels)
    int chunks;         // total chunks of the reduction
    int a_sub_px;       // pixels per A box = min(64, PQ)
    int a_subs;         // A boxes per chunk
    int a_sub_bytes;    // kb * a_sub_px * 2
    int a_region_bytes; // a_subs * a_sub_bytes rounded up to 1 KiB (B tiles start there)
    int a_swz, b_swz;   // swizzle codes of the descriptors
    int b_tiles;        // S (halo) or R*S
    int b_tile_stride;  // bytes between consecutive B tiles (multiple of 1024)
    int b_tile_bytes;   // bytes one TMA writes per B tile
    int stage_bytes, stages;
    int ksteps;         // ci*bp*Q/16
    int tmem_cols;      // power of two >= 32
    uint32_t idesc;
};

constexpr int kMaxStages = 8;

__global__ void __launch_bounds__(192, 1)
exact_tc_kernel(const __grid_constant__ CUtensorMap map_dy, const __grid_constant__ CUtensorMap map_x,
                float* __restrict__ dw, float* __restrict__ partial, uint32_t* __restrict__ counters,
                uint32_t* __restrict__ status, const TcParams P)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bar_full[kMaxStages], bar_empty[kMaxStages], bar_acc;
    __shared__ uint32_t s_tmem_base;
    __shared__ volatile int s_abort;
    __shared__ bool s_last;

    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Geom& g = P.g;

    const int tile = blockIdx.x, split = blockIdx.y;
    const int k0 = (tile / P.tiles_c) * P.m, c0 = (tile % P.tiles_c) * P.ct;
    const int per = (P.chunks + P.splits - 1) / P.splits;
    const int ch_begin = min(P.chunks, split * per), ch_end = min(P.chunks, ch_begin + per);
    const int nchunks = ch_end - ch_begin;
    const int nmma = g.s * P.ct;

    if (threadIdx.x == 0) {
        for (int i = 0; i < P.stages; ++i) { mbar_init(smem_u32(&bar_full[i]), 1); mbar_init(smem_u32(&bar_empty[i]), 1); }
        mbar_init(smem_u32(&bar_acc), 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)), "r"(P.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = s_tmem_base;

    if (warp == 0 && lane == 0) {
        // ------------------------------------------------------------------ TMA producer
        int issued = 0;
        for (int it = 0; it < nchunks; ++it) {
            const int st = it % P.stages;
            if (it >= P.stages && !mbar_wait(smem_u32(&bar_empty[st]), ((it / P.stages) - 1) & 1)) { s_abort = 1; atomicOr(status, 1u); break; }
            if (s_abort) break;
            const int ch = ch_begin + it;
            const uint32_t full = smem_u32(&bar_full[st]);
            const uint32_t sa = smem_base + st * P.stage_bytes;
            const uint32_t sb = sa + P.a_region_bytes;
            mbar_expect_tx(full, P.a_subs * P.a_sub_bytes + P.b_tiles * P.b_tile_bytes);
            int n0, p0;
            if (P.ci > 1 || P.a_sub_px < 64) { n0 = ch * P.ci; p0 = 0; }
            else { const int cpi = g.p / P.bp; n0 = ch / cpi; p0 = (ch % cpi) * P.bp; }
            if (P.a_sub_px < 64) {
                tma_load_3d(sa, &map_dy, full, 0, k0, n0);                       // ci whole maps in one box
            } else {
                for (int b = 0; b < P.a_subs; ++b) tma_load_3d(sa + b * P.a_sub_bytes, &map_dy, full, p0 * g.q + 64 * b, k0, n0);
            }
            for (int t = 0; t < P.b_tiles; ++t) {
                const int s = t % g.s, r = t / g.s;
                const int h0 = P.halo ? p0 - g.pad_h : p0 * g.stride_h + r - g.pad_h;
                tma_load_4d(sb + t * P.b_tile_stride, &map_x, full, c0, s - g.pad_w, h0, n0);
            }
            ++issued;
        }
        if (s_abort) {   // drain: wait (bounded) for the copies already issued
            for (int it = max(0, issued - P.stages); it < issued; ++it) mbar_wait(smem_u32(&bar_full[it % P.stages]), (it / P.stages) & 1);
        }
    } else if (warp == 1 && lane == 0) {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t a_row_bytes = P.a_sub_px * 2, a_sbo = 8 * a_row_bytes;
        const uint32_t b_row_bytes = P.ct * 2, b_sbo = 8 * b_row_bytes;
        const int ks_per_sub = P.a_sub_px / 16;
        bool ok = true;
        for (int it = 0; it < nchunks && ok; ++it) {
            const int st = it % P.stages;
            if (!mbar_wait(smem_u32(&bar_full[st]), (it / P.stages) & 1)) { s_abort = 1; atomicOr(status, 1u); ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t sa = smem_base + st * P.stage_bytes;
            const uint32_t sb = sa + P.a_region_bytes;
            for (int kk = 0; kk < P.ksteps; ++kk) {
                const uint64_t adesc = smem_desc(sa + (kk / ks_per_sub) * P.a_sub_bytes + (kk % ks_per_sub) * 32, 16, a_sbo, P.a_swz);
                for (int r = 0; r < g.r; ++r) {
                    const uint32_t baddr = sb + (P.halo ? 0 : r * g.s * P.b_tile_stride) + (16 * kk + (P.halo ? r * g.q : 0)) * b_row_bytes;
                    const uint64_t bdesc = smem_desc(baddr, P.b_tile_stride, b_sbo, P.b_swz);
                    const uint32_t d = P.m == 128 ? tmem_base + r * nmma : tmem_base + (((uint32_t)(r & 1) * 16u) << 16) + (r >> 1) * nmma;
                    umma_bf16(d, adesc, bdesc, P.idesc, (it > 0 || kk > 0) ? 1u : 0u);
                }
            }
            umma_commit(smem_u32(&bar_empty[st]));   // frees the stage once these MMAs have read it
        }
        umma_commit(smem_u32(&bar_acc));             // accumulators complete
    } else if (warp >= 2) {
        // ------------------------------------------------------------------ epilogue: TMEM -> global
        const bool ready = mbar_wait(smem_u32(&bar_acc), 0);
        if (!ready) { s_abort = 1; atomicOr(status, 1u); }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ready && !s_abort) {
            const int sp = warp & 3;
            float* out = P.splits == 1 ? dw : partial + (size_t)split * g.k * g.r * g.s * g.c;
            const float scale = P.splits == 1 ? g.alpha : 1.0f;
            const int groups = P.m == 128 ? g.r : (g.r + 1) / 2;
            for (int gi = 0; gi < groups; ++gi) {
                const int r = P.m == 128 ? gi : 2 * gi + (lane >> 4);
                const int k = k0 + (P.m == 128 ? 32 * sp + lane : 16 * sp + (lane & 15));
                const bool row_ok = r < g.r && k < g.k && (nchunks > 0 || true);
                for (int j0 = 0; j0 < nmma; j0 += 16) {
                    float v[16];
                    const uint32_t taddr = tmem_base + ((uint32_t)(32 * sp) << 16) + gi * nmma + j0;
                    if (nmma - j0 >= 16) tmem_ld16(taddr, v); else tmem_ld8(taddr, v);
                    if (!row_ok) continue;
                    const int lim = min(16, nmma - j0);
                    for (int jj = 0; jj < lim; ++jj) {
                        const int nn = j0 + jj, s = nn / P.ct, c = c0 + nn % P.ct;
                        if (c < g.c) out[k * g.ws_k + c * g.ws_c + r * g.ws_r + s * g.ws_s] = nchunks > 0 ? scale * v[jj] : 0.0f;
                    }
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(P.tmem_cols) : "memory");
    }
    if (P.splits == 1 || s_abort) return;

    // ---------------------------------------------------------------------- split reduction (last CTA of the tile)
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(&counters[tile % kWsNumCounters], 1u) == (uint32_t)P.splits - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const int rows = min(P.m, g.k - k0), cols = min(P.ct, g.c - c0);
    const int per_row = g.r * g.s * cols;
    const size_t kcrs = (size_t)g.k * g.r * g.s * g.c;
    for (int e = threadIdx.x; e < rows * per_row; e += blockDim.x) {
        const int kk = e / per_row, rem = e % per_row;
        const int r = rem / (g.s * cols), s = (rem / cols) % g.s, c = c0 + rem % cols;
        const size_t off = (k0 + kk) * g.ws_k + c * g.ws_c + r * g.ws_r + s * g.ws_s;
        float tot = 0.f;
        for (int sp = 0; sp < P.splits; ++sp) tot += __ldcg(partial + sp * kcrs + off);
        dw[off] = g.alpha * tot;
    }
    if (threadIdx.x == 0) counters[tile % kWsNumCounters] = 0;
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

CUtensorMapSwizzle swizzle_for(int bytes) {
    return bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
}
int swz_code(int bytes) { return bytes == 128 ? 2 : bytes == 64 ? 4 : 6; }
int pow2_ceil(int v) { int p = 32; while (p < v) p *= 2; return p; }
int env_int(const char* name, int dflt) { const char* e = getenv(name); return e ? atoi(e) : dflt; }

}  // namespace

bool plan_tc(const Geom& g, TcPlan* out)
{
    if (!g.bf16) return false;
    if (g.xs_c != 1 || g.c % 8 != 0) return false;                       // NHWC with 16-byte pixel rows
    if (g.stride_h != g.stride_w) return false;
    const int pq = g.p * g.q;
    if (pq % 16 != 0 || (pq < 64 && pq != 16 && pq != 32) || (pq >= 64 && pq % 64 != 0)) return false;
    const bool small_map = pq < 64;
    const bool halo = !small_map && g.stride_h == 1 && g.q % 8 == 0 && 64 % g.q == 0;
    if (!small_map && !(g.q <= 64 && 64 % g.q == 0)) return false;        // a 64-pixel box must be whole rows
    if (g.r > 7 || g.s > 7) return false;

    TcParams P{};
    P.g = g;
    P.m = g.k <= 64 ? 64 : 128;
    P.kb = (g.k < P.m ? (g.k + 7) / 8 * 8 : P.m);
    // channels per tile: one swizzle span wide (16, 32 or 64 channels), limited by MMA N <= 256 and TMEM columns
    int ct = g.c >= 64 ? 64 : g.c >= 32 ? 32 : 16;
    auto cols_for = [&](int c) { return (P.m == 128 ? g.r : (g.r + 1) / 2) * g.s * c; };
    while (ct > 16 && (g.s * ct > 256 || cols_for(ct) > 512)) ct /= 2;
    if (g.s * ct > 256 || cols_for(ct) > 512) return false;
    if ((g.s * ct) % (P.m == 128 ? 16 : 8) != 0) return false;
    P.ct = ct;
    P.tiles_k = (g.k + P.m - 1) / P.m;
    P.tiles_c = (g.c + ct - 1) / ct;
    if (P.tiles_k * P.tiles_c > kWsNumCounters) return false;
    P.halo = halo ? 1 : 0;
    P.a_sub_px = small_map ? pq : 64;
    P.a_swz = swz_code(P.a_sub_px * 2);
    P.b_swz = swz_code(ct * 2);
    P.b_tiles = halo ? g.s : g.r * g.s;

    // chunk size: as many rows (or images) as fit a ~48 KiB stage
    const int budget = env_int("GACONV_TC_STAGE_KB", 48) * 1024;
    auto stage_bytes = [&](int ci, int bp, int* a_subs, int* tile_bytes, int* tile_stride) {
        const int px = ci * bp * g.q;
        *a_subs = small_map ? ci : px / 64;
        const int a_bytes = ((small_map ? P.kb * pq * 2 * ci : *a_subs * P.kb * 128) + 1023) / 1024 * 1024;
        const int rows = halo ? bp + g.r - 1 : bp;
        *tile_bytes = ci * rows * g.q * ct * 2;
        *tile_stride = (*tile_bytes + 1023) / 1024 * 1024;
        return a_bytes + P.b_tiles * *tile_stride;
    };
    int ci = 1, bp = small_map ? g.p : 64 / g.q, a_subs, tb, ts;
    if (small_map) {
        while (ci * 2 <= 16 && ci * 2 <= g.n && stage_bytes(ci * 2, bp, &a_subs, &tb, &ts) <= budget) ci *= 2;
    } else {
        while (bp * 2 <= g.p && g.p % (bp * 2) == 0 && (halo ? bp * 2 + g.r - 1 : bp * 2 * g.stride_h) <= 256 &&
               stage_bytes(1, bp * 2, &a_subs, &tb, &ts) <= budget) bp *= 2;
        if (g.p % bp != 0) return false;
    }
    P.ci = ci; P.bp = bp;
    P.stage_bytes = stage_bytes(ci, bp, &a_subs, &tb, &ts);
    P.stage_bytes = (P.stage_bytes + 1023) / 1024 * 1024;
    P.a_subs = a_subs; P.b_tile_bytes = tb; P.b_tile_stride = ts;
    P.a_sub_bytes = small_map ? P.kb * pq * 2 : P.kb * 128;   // small maps: per image; one box carries ci of them
    P.a_region_bytes = (P.a_subs * P.a_sub_bytes + 1023) / 1024 * 1024;
    P.ksteps = ci * bp * g.q / 16;
    P.chunks = small_map ? (g.n + ci - 1) / ci : g.n * (g.p / bp);
    const int smem_budget = 200 * 1024;
    P.stages = smem_budget / P.stage_bytes;
    if (P.stages > kMaxStages) P.stages = kMaxStages;
    if (P.stages < 2) return false;
    P.tmem_cols = pow2_ceil(cols_for(ct));
    if (P.tmem_cols > 512) return false;
    // instruction descriptor: fp32 accumulate, bf16 x bf16, A K-major, B MN-major, N, M
    P.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) | ((uint32_t)(g.s * ct >> 3) << 17) | ((uint32_t)(P.m >> 4) << 24);

    const int tiles = P.tiles_k * P.tiles_c;
    int splits = env_int("GACONV_TC_SPLITS", 0);
    if (splits <= 0) {
        splits = 148 / tiles;
        if (splits < 1) splits = 1;
        // partial blocks are written and read back: keep them well below the input bytes
        const size_t out_bytes = (size_t)g.k * g.r * g.s * g.c * 4;
        const size_t in_bytes = ((size_t)g.n * g.c * g.h * g.w + (size_t)g.n * g.k * pq) * 2;
        while (splits > 1 && (size_t)splits * out_bytes > in_bytes / 2 + (1 << 20)) --splits;
    }
    if (splits > P.chunks) splits = P.chunks;
    {   // no empty splits: every CTA gets ceil(chunks / splits) chunks except possibly the last
        const int per = (P.chunks + splits - 1) / splits;
        splits = (P.chunks + per - 1) / per;
    }
    P.splits = splits;

    out->partial_bytes = splits > 1 ? (size_t)splits * g.k * g.r * g.s * g.c * 4 : 0;
    static_assert(sizeof(TcParams) <= sizeof(out->opaque), "TcPlan::opaque too small");
    memcpy(out->opaque, &P, sizeof(P));
    return encode_fn() != nullptr;
}

cudaError_t launch_tc(const void* x, const void* dy, float* dw, float* partial, uint32_t* counters, uint32_t* status,
                      const TcPlan& plan, cudaStream_t stream)
{
    TcParams P;
    memcpy(&P, plan.opaque, sizeof(P));
    const Geom& g = P.g;
    const int pq = g.p * g.q;
    EncodeTiledFn enc = encode_fn();
    if (enc == nullptr) return cudaErrorNotSupported;

    CUtensorMap map_dy, map_x;
    {   // dY as (pq, k, n), bf16
        cuuint64_t dims[3] = {(cuuint64_t)pq, (cuuint64_t)g.k, (cuuint64_t)g.n};
        cuuint64_t strides[2] = {(cuuint64_t)pq * 2, (cuuint64_t)g.k * pq * 2};
        cuuint32_t box[3] = {(cuuint32_t)P.a_sub_px, (cuuint32_t)P.kb, (cuuint32_t)(P.a_sub_px < 64 ? P.ci : 1)};
        cuuint32_t es[3] = {1, 1, 1};
        if (enc(&map_dy, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(dy), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(P.a_sub_px * 2), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    {   // X as (c, w, h, n), bf16; a box is ct channels x q columns x rows x ci images, stepping by the conv stride
        cuuint64_t dims[4] = {(cuuint64_t)g.c, (cuuint64_t)g.w, (cuuint64_t)g.h, (cuuint64_t)g.n};
        cuuint64_t strides[3] = {(cuuint64_t)g.c * 2, (cuuint64_t)g.w * g.c * 2, (cuuint64_t)g.h * g.w * g.c * 2};
        const int rows = P.halo ? P.bp + g.r - 1 : P.bp;
        cuuint32_t box[4] = {(cuuint32_t)P.ct, (cuuint32_t)(g.q * g.stride_w), (cuuint32_t)(rows * g.stride_h), (cuuint32_t)P.ci};
        cuuint32_t es[4] = {1, (cuuint32_t)g.stride_w, (cuuint32_t)g.stride_h, 1};
        if (enc(&map_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(x), dims, strides, box, es,
                CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(P.ct * 2), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    // dynamic shared memory: stages, 1 KiB of alignment slack, and a tail so that the MMA's read of
    // all M rows of an A box with fewer valid rows stays inside the allocation
    const size_t smem = (size_t)P.stages * P.stage_bytes + 1024 + (size_t)P.m * 128;
    static size_t configured = 0;
    if (smem > configured) {
        cudaError_t e = cudaFuncSetAttribute(exact_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured = smem;
    }
    dim3 grid(P.tiles_k * P.tiles_c, P.splits);
    exact_tc_kernel<<<grid, 192, smem, stream>>>(map_dy, map_x, dw, partial, counters, status, P);
    note_launch();
    return cudaGetLastError();
}

}  // namespace gaconv
